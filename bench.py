#!/usr/bin/env python
"""Benchmark of the batched tree-verification attention (Sec. 3.2) and of the step around it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

The headline is verify attention alone: `value` is verified tree-tokens per second of one
reader_verify_attn call (batch * tree nodes / call time; ancestor masks encoded beforehand) with
every input resident in HBM, and `roofline` is that call's attention kernel against the measured
HBM copy bandwidth (or the measured bf16 tensor throughput where that binds).  A timed block is K
calls; blocks are repeated until about a second has been timed and the median block is reported.
`e2e` is the same call with the step's inputs (Q, tree K/V, parent arrays) copied from pinned host
memory and the output copied back inside the timed region.  `workloads` holds the same
measurement, L2 flushed before every call, for all five workloads C1..C5.  The acceptance (target
argmax + walk) and the KV commit are timed separately (`kernels`), and the whole step
(attention + acceptance + commit), a 32-layer model step and the side kernels are reported in
keys of their own, never folded into the attention number.  Sequences are independent, so N GPUs
run N replicas of the batch with no data-path collective (weak scaling).  Prints one JSON line on
rank 0.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import re
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified tree-tokens/sec and achieved HBM GB/s (% of B200 peak), verify attn, 1 GPU"
UNIT = "tokens/s"
LAUNCHES_PER_ATTN_CALL = 3   # preparation, attention, combine
LAUNCHES_PER_STEP = 5        # + argmax, acceptance walk with commit
L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# ncu counters of one launch are kept as text under profiles/; each summary records the SHA-256 of the
# kernel sources it was taken from, and a figure is used only while those sources are unchanged.
TRAFFIC_PROFILES = {("verify_attn", "c3"): "attn_sm100_c3.md", ("argmax", "c3"): "argmax_c3.md"}
TRAFFIC_SOURCES = {"verify_attn": ("verify_attn_sm100.cu", "common.cuh", "ptx_sm100.cuh"), "argmax": ("accept.cu",)}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def source_digest(kind: str) -> str:
    h = hashlib.sha256()
    for f in TRAFFIC_SOURCES[kind]:
        h.update(open(os.path.join(ROOT, "paper_2508_09072_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(kind: str, workload: str):
    """(bytes per launch, where from) out of the profile summary, or (None, why): the summary names the
    digest of the sources its counters were taken from."""
    name = TRAFFIC_PROFILES.get((kind, workload))
    if not name:
        return None, "no ncu capture of this workload"
    try:
        text = open(os.path.join(ROOT, "profiles", name)).read()
        m_b = re.search(r"^traffic-bytes-per-launch:\s*([0-9.eE+]+)", text, re.M)
        m_s = re.search(r"^source-sha256-16:\s*([0-9a-f]{16})", text, re.M)
        m_c = re.search(r"^captured-at-commit:\s*(\S+)", text, re.M)
        if not (m_b and m_s):
            return None, f"profiles/{name} states no counters"
        if m_s.group(1) != source_digest(kind):
            return None, f"kernel sources changed since the capture in profiles/{name}"
        return float(m_b.group(1)), f"ncu capture in profiles/{name} (commit {m_c.group(1) if m_c else '?'}), not this run"
    except OSError:
        return None, f"profiles/{name} missing"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.06] or [l for (_, l) in self.lines[-3:]]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except Exception:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def fits_l2(w) -> bool:
    return w.attn_algorithmic_bytes() <= 2 * L2_BYTES


def workload_config(w, name):
    import numpy as np
    return {"workload": name, "batch": int(w.batch), "tree_nodes": int(w.n_nodes), "n_q_heads": int(w.n_q_heads),
            "n_kv_heads": int(w.n_kv_heads), "head_dim": int(w.head_dim), "page_size": int(w.page_size),
            "committed_tokens": int(np.sum(w.seq_lens)), "shared_prefix_len": int(w.shared_prefix_len),
            "l2": ("L2 flushed before every call (a read pass over 512 MB): the call's inputs fit the 126 MB L2" if fits_l2(w)
                   else "no flush: every call streams more K/V than the 126 MB L2 holds")}


def median(xs):
    xs = sorted(xs)
    return xs[len(xs) // 2]


# ------------------------------------------------------------------------------------------------
# CPU baseline: the checker as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------
def one_sequence(w, b):
    """Sequence b of the workload as a batch of one (views; the pool is shared)."""
    import copy
    s = copy.copy(w)
    s.batch = 1
    for f in ("q", "k_tree", "v_tree", "parent", "node_tokens", "logits"):
        if getattr(w, f) is not None:
            setattr(s, f, getattr(w, f)[b:b + 1])
    s.page_table, s.seq_lens = w.page_table[b:b + 1], w.seq_lens[b:b + 1]
    return s


def cpu_attn_sample(w, seqs):
    """The CPU checker's verify attention on the given sequences of the workload; returns seconds."""
    import oracle
    t0 = time.perf_counter()
    for b in seqs:
        s = one_sequence(w, b)
        oracle.verify_attn(s.q, s.k_tree, s.v_tree, w.k_pool, w.v_pool, s.page_table, s.seq_lens, s.parent, w.scale)
    return time.perf_counter() - t0


def cpu_step_sample(w, seqs):
    """The CPU checker's whole step (attention, argmax, acceptance, commit) on the given sequences; seconds."""
    import numpy as np
    import oracle
    t0 = time.perf_counter()
    for b in seqs:
        s = one_sequence(w, b)
        oracle.verify_attn(s.q, s.k_tree, s.v_tree, w.k_pool, w.v_pool, s.page_table, s.seq_lens, s.parent, w.scale)
        tgt = oracle.argmax(s.logits)
        a = oracle.accept(s.parent, s.node_tokens, tgt, w.max_path)
        # commit on the sequence's own pages only (the checker copies the pool it is given)
        used = s.page_table[0][s.page_table[0] >= 0]
        remap = np.full(w.num_pages, -1, np.int32)
        remap[used] = np.arange(len(used), dtype=np.int32)
        pt = np.where(s.page_table >= 0, remap[np.maximum(s.page_table, 0)], -1).astype(np.int32)
        oracle.kv_commit(w.k_pool[used], w.v_pool[used], pt, s.seq_lens, 0, s.k_tree, s.v_tree, a["path"], a["n_acc"])
    return time.perf_counter() - t0


def cpu_baseline(w, budget_s=12.0):
    """The checker as it stands: verify attention, sequence after sequence (wrapping around the batch),
    until about budget_s seconds of CPU work are done; then a few whole steps for the step's figure."""
    import oracle
    cores = oracle.num_threads()
    done, spent = 0, 0.0
    while spent < budget_s and done < 64 * w.batch:
        spent += cpu_attn_sample(w, [done % w.batch])
        done += 1
    res = {"value": done * w.n_nodes / spent, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"verify attention on {done} sequences drawn in order from the {w.batch} of the workload "
                     f"({done * w.n_nodes} tree tokens), {spent:.1f} s"}
    if w.logits is not None:
        n, t = 0, 0.0
        while t < 3.0 and n < w.batch:
            t += cpu_step_sample(w, [n])
            n += 1
        res["whole_step"] = {"value": n * w.n_nodes / t, "unit": UNIT,
                             "sample": f"attention + argmax + acceptance + commit on {n} sequences, {t:.1f} s"}
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2508_09072_b200 import workloads as W
    oracle.build()
    w = W.make(args.workload, with_logits=False)
    t1 = cpu_attn_sample(w, [0])                      # also warms the page cache and the library
    per_step = 120.0 / (args.steps + args.warmup)     # the whole run should end within a few minutes
    n_seq = int(min(w.batch, max(1, per_step / max(t1, 1e-4))))
    seqs = list(range(n_seq))
    for _ in range(args.warmup):
        cpu_attn_sample(w, seqs)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        cpu_attn_sample(w, seqs)
    dt = time.perf_counter() - t0
    value = args.steps * n_seq * w.n_nodes / dt
    cores = oracle.num_threads()
    sample = f"each step = verify attention on the first {n_seq} of {w.batch} sequences of {args.workload}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, args.workload),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------------
# N > 1: independent replicas (sequences do not interact), no data-path collective
# ------------------------------------------------------------------------------------------------
def max_over_ranks(values, device, world):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the time)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_tokens_per_s(batch, tree_nodes, world, steps, ms_max):
    """Whole-job throughput: every rank verified batch * tree_nodes tokens per step; the job took the
    time of its slowest rank."""
    return batch * tree_nodes * world * steps / (ms_max * 1e-3)


def blocks_for(t_call_ms: float, steps: int, target_ms: float, cap_calls: int) -> int:
    """How many blocks of `steps` calls to time so that about target_ms of device time is covered."""
    per_block = max(t_call_ms * steps, 1e-6)
    return int(max(1, min(math.ceil(target_ms / per_block), max(1, cap_calls // max(steps, 1)))))


# ------------------------------------------------------------------------------------------------
# verify attention of one workload: kernel alone, isolated call, back-to-back calls
# ------------------------------------------------------------------------------------------------
class AttnCase:
    """One workload on the device with everything a reader_verify_attn call needs."""

    def __init__(self, rd, w, dev, with_logits=False):
        import torch
        from paper_2508_09072_b200 import binding
        self.rd, self.w = rd, w
        self.d = d = binding.to_device(w, dev, with_logits=with_logits)
        self.anc, _, enc_status = rd.tree_encode(d.parent)
        self.out = torch.empty_like(d.q)
        self.status = torch.empty(w.batch, dtype=torch.int32, device=dev)
        self.ws = rd.workspace(w.batch, w.n_nodes, w.n_q_heads, w.n_kv_heads, w.head_dim)
        assert int(enc_status.max().item()) == 0

    def call(self):
        d = self.d
        self.rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, self.w.scale, anc_mask=self.anc, out=self.out,
                            status=self.status, workspace=self.ws)


def attn_row(case: AttnCase, flush, peaks, iters: int, pipelined_ms: float):
    """Cold-L2 figures of one workload: the attention kernel alone (events inside the call) and the whole
    call (events around it, its launches overlapping as in production); optionally back-to-back calls."""
    import torch
    rd, w = case.rd, case.w
    mk = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(5):
        case.call()
    tk, tc = [], []
    for _ in range(iters):
        flush()
        c, e = mk(), mk()
        c.record(); e.record()
        rd.set_timing_events(c, e)
        case.call()
        torch.cuda.synchronize()
        tk.append(c.elapsed_time(e))
    rd.set_timing_events(None, None)
    for _ in range(iters):
        flush()
        a, b = mk(), mk()
        a.record(); case.call(); b.record()
        torch.cuda.synchronize()
        tc.append(a.elapsed_time(b))
    assert int(case.status.max().item()) == 0
    k, c_ = median(tk) * 1e-3, median(tc) * 1e-3
    by, fl = w.attn_algorithmic_bytes(), w.attn_algorithmic_flops()
    t_hbm, t_tc = by / (peaks["hbm_gbs"] * 1e9), fl / (peaks["bf16_tflops_sustained"] * 1e12)
    row = {"workload": w.name, "tokens": w.batch * w.n_nodes, "kernel_us": k * 1e6, "kernel_us_min": min(tk) * 1e3,
           "call_us": c_ * 1e6, "call_us_min": min(tc) * 1e3, "algorithmic_bytes": by, "algorithmic_flops": fl,
           "gbs": by / k / 1e9, "hbm_frac": by / k / 1e9 / peaks["hbm_gbs"], "hbm_frac_of_nominal_8tbs": by / k / 8e12,
           "tflops": fl / k / 1e12, "tensor_frac": fl / k / 1e12 / peaks["bf16_tflops_sustained"],
           "t_hbm_us": t_hbm * 1e6, "t_tensor_us": t_tc * 1e6,
           "binding_bound": "hbm" if t_hbm >= t_tc else "tensor", "binding_frac": max(t_hbm, t_tc) / k,
           "binding_frac_call": max(t_hbm, t_tc) / c_, "tokens_per_s": w.batch * w.n_nodes / c_,
           "l2": "flushed before every call"}
    if pipelined_ms > 0 and not fits_l2(w):
        n = max(20, int(pipelined_ms / (c_ * 1e3)))
        a, b = mk(), mk()
        a.record()
        for _ in range(n):
            case.call()
        b.record()
        torch.cuda.synchronize()
        row["call_us_back_to_back"] = a.elapsed_time(b) / n * 1e3
        row["tokens_per_s_back_to_back"] = w.batch * w.n_nodes / (a.elapsed_time(b) / n * 1e-3)
    return row


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2508_09072_b200 import binding, workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    peaks, peak_kind = load_peaks()

    w = W.make(args.workload, seed_offset=rank)
    rd = binding.Reader(local)
    if args.kernel:
        rd.set_attn_kernel(args.kernel)
    case = AttnCase(rd, w, dev, with_logits=True)
    d, out, status, ws = case.d, case.out, case.status, case.ws
    B, T = w.batch, w.n_nodes
    K, Wm = args.steps, max(args.warmup, 3)
    small = fits_l2(w)
    flush_buf = torch.zeros((512 << 20) // 4, dtype=torch.int32, device=dev)
    flush_sink = torch.zeros((), dtype=torch.int64, device=dev)

    def flush():
        # a READ pass over four times the L2: the cache ends up holding clean lines of a buffer nobody
        # uses (a write pass would leave 126 MB of dirty lines to be written back under the next kernel)
        torch.sum(flush_buf, dim=(0,), out=flush_sink)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def mk():
        return torch.cuda.Event(enable_timing=True)

    # ---- main region: blocks of K reader_verify_attn calls, device-resident inputs
    for _ in range(Wm):
        case.call()
    p0, p1 = mk(), mk()
    torch.cuda.synchronize()
    p0.record()
    for _ in range(10):
        case.call()
    p1.record()
    torch.cuda.synchronize()
    t_est = p0.elapsed_time(p1) / 10
    n_blocks = blocks_for(t_est, K, args.min_timed_ms if not small else args.min_timed_ms / 4, 40000 if not small else 8000)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    t_wall0 = time.time()
    if not small:
        marks = [mk() for _ in range(n_blocks + 1)]
        marks[0].record()
        for i in range(n_blocks):
            for _ in range(K):
                case.call()
            marks[i + 1].record()
        barrier()
        block_ms = [marks[i].elapsed_time(marks[i + 1]) for i in range(n_blocks)]
    else:
        pairs = [(mk(), mk()) for _ in range(n_blocks * K)]
        for a, b in pairs:
            flush()
            a.record(); case.call(); b.record()
        barrier()
        ts = [a.elapsed_time(b) for a, b in pairs]
        block_ms = [sum(ts[i * K:(i + 1) * K]) for i in range(n_blocks)]
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_block = median(block_ms)
    assert int(status.max().item()) == 0

    # ---- the attention kernel alone: a second loop with events inside the call around the kernel (events
    # between two kernels switch the overlap of their launches off, so this loop is a little slower)
    Kb = max(20, min(300, n_blocks * K))
    kev = [(mk(), mk()) for _ in range(Kb)]
    for a, b in kev:                                  # create the handles
        a.record(); b.record()
    worst = torch.zeros((), dtype=torch.int32, device=dev)   # a bounded wait that gave up shows in the status words
    for i in range(Kb):
        if small:
            flush()
        rd.set_timing_events(*kev[i])
        case.call()
        worst = torch.maximum(worst, status.max())
    barrier()
    rd.set_timing_events(None, None)
    assert int(worst.item()) == 0, f"status {int(worst.item())} seen during the kernel-timing loop"
    t_attn_kernel = sum(a.elapsed_time(b) for a, b in kev) / Kb

    # ---- end to end: the step's inputs from pinned host memory, the output back, every call
    host_in = {k: getattr(d, k).cpu().pin_memory() for k in ("q", "k_tree", "v_tree", "parent")}
    host_out = {"out": torch.empty(out.shape, dtype=out.dtype).pin_memory(),
                "status": torch.empty(B, dtype=torch.int32).pin_memory()}
    h2d = sum(t.numel() * t.element_size() for t in host_in.values())
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())

    def e2e_call():
        for k, t in host_in.items():
            getattr(d, k).copy_(t, non_blocking=True)
        rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, out=out, status=status, workspace=ws)
        host_out["out"].copy_(out, non_blocking=True)
        host_out["status"].copy_(status, non_blocking=True)
        torch.cuda.current_stream().synchronize()     # the caller needs the result before the next step

    for _ in range(3):
        e2e_call()
    q0, q1 = mk(), mk()
    q0.record(); e2e_call(); q1.record()
    torch.cuda.synchronize()
    ne = blocks_for(q0.elapsed_time(q1), K, args.min_timed_ms / 4, 4000)
    barrier()
    e_ms = []
    for _ in range(ne):
        f0, f1 = mk(), mk()
        f0.record()
        for _ in range(K):
            e2e_call()
        f1.record()
        torch.cuda.synchronize()
        e_ms.append(f0.elapsed_time(f1))
    barrier()
    ms_e2e_block = median(e_ms)
    assert int(host_out["status"].max().item()) == 0

    # ---- the whole step: attention (masks encoded inside the call), acceptance from logits, commit
    seq_lens0 = d.cache.seq_lens.clone()
    tgt = torch.empty((B, T), dtype=torch.int32, device=dev)
    acc_out = (torch.empty((B, w.max_path), dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev),
               torch.empty(B, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev))
    slots = torch.empty((B, w.max_path), dtype=torch.int32, device=dev)
    cstat = torch.empty(B, dtype=torch.int32, device=dev)

    def step(ev=None):
        d.cache.seq_lens.copy_(seq_lens0)            # harness: rewind the cache length
        if ev:
            ev[0].record()
        rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, out=out, status=status, workspace=ws)
        if ev:
            ev[1].record()
        rd.accept_commit(d.parent, d.node_tokens, w.max_path, d.cache, d.k_tree, d.v_tree, logits=d.logits, target_ids=tgt,
                         workspace=ws, outs=acc_out, slots=slots, commit_status=cstat)
        if ev:
            ev[2].record()

    for _ in range(3):
        step()
    Ks = max(20, min(300, n_blocks * K))
    s0, s1 = mk(), mk()
    barrier()
    s0.record()
    for _ in range(Ks):
        step()
    s1.record()
    barrier()
    t_step = s0.elapsed_time(s1) / Ks
    assert int(status.max().item()) == 0 and int(cstat.max().item()) == 0 and int(acc_out[3].max().item()) == 0
    evs = [[mk() for _ in range(3)] for _ in range(Ks)]
    aev = [(mk(), mk()) for _ in range(Ks)]
    for a, b in aev:
        a.record(); b.record()
    for i in range(Ks):
        rd.set_accept_timing_events(*aev[i])
        step(evs[i])
    barrier()
    rd.set_accept_timing_events(None, None)
    t_attn_in_step = sum(e[0].elapsed_time(e[1]) for e in evs) / Ks
    t_accept = sum(e[1].elapsed_time(e[2]) for e in evs) / Ks
    t_argmax_kernel = sum(a.elapsed_time(b) for a, b in aev) / Ks

    # reader_kv_commit on its own (the step above runs it inside reader_accept_commit)
    c_times = []
    for _ in range(20):
        d.cache.seq_lens.copy_(seq_lens0)
        c0, c1 = mk(), mk()
        c0.record()
        rd.kv_commit(d.cache, d.k_tree, d.v_tree, acc_out[0], acc_out[1], slots=slots, status=cstat)
        c1.record()
        torch.cuda.synchronize()
        c_times.append(c0.elapsed_time(c1))
    t_commit = median(c_times)
    # and the acceptance walk alone, from given target ids
    a_times = []
    for _ in range(20):
        a0, a1 = mk(), mk()
        a0.record()
        rd.accept(d.parent, d.node_tokens, w.max_path, target_ids=tgt, outs=acc_out)
        a1.record()
        torch.cuda.synchronize()
        a_times.append(a0.elapsed_time(a1))
    t_walk = median(a_times)

    extras = {}
    if not args.quick:
        extras = run_extras(args, rd, w, d, dev, rank, step, seq_lens0, out, status, ws, tgt, acc_out, slots, cstat, barrier, mk)

    # ---- all five workloads, L2 flushed before every call (rank 0 of a single-GPU run)
    table = None
    if world == 1 and not args.no_table:
        table = []
        for name in W.WORKLOADS:
            if name == args.workload:
                c2 = case
            else:
                c2 = AttnCase(rd, W.make(name, with_logits=False), dev)
            table.append(attn_row(c2, flush, peaks, args.table_iters, 30.0))
            if c2 is not case:
                del c2
                torch.cuda.empty_cache()

    long_prefix = None
    if world == 1 and not args.no_table:
        long_prefix = long_prefix_rows(rd, dev, peaks, args.table_iters)

    # ---- max over ranks
    ms_block, ms_e2e_block, t_attn_kernel, t_step, t_accept, t_argmax_kernel, t_commit, t_walk = max_over_ranks(
        [ms_block, ms_e2e_block, t_attn_kernel, t_step, t_accept, t_argmax_kernel, t_commit, t_walk], dev, world)

    if rank == 0:
        tokens = B * T * world
        value = aggregate_tokens_per_s(B, T, world, K, ms_block)
        e2e = aggregate_tokens_per_s(B, T, world, K, ms_e2e_block)
        attn_bytes, attn_flops = w.attn_algorithmic_bytes(), w.attn_algorithmic_flops()
        t_call = ms_block / K
        t_hbm = attn_bytes / (peaks["hbm_gbs"] * 1e9)
        t_tc = attn_flops / (peaks["bf16_tflops_sustained"] * 1e12)
        bound = "hbm" if t_hbm >= t_tc else "tensor"
        gbs = attn_bytes / (t_attn_kernel * 1e-3) / 1e9
        tfs = attn_flops / (t_attn_kernel * 1e-3) / 1e12
        traffic, traffic_src = ncu_traffic("verify_attn", args.workload)
        if bound == "hbm":
            roof = {"kernel": "verify_attn (attn_sm100_kernel)", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": traffic, "traffic_source": traffic_src,
                    "peak_kind": peak_kind, "frac_of_nominal_8tbs": gbs / 8000.0,
                    "frac_whole_call": attn_bytes / (t_call * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        else:
            roof = {"kernel": "verify_attn (attn_sm100_kernel)", "bound": "tensor", "achieved": tfs,
                    "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": tfs / peaks["bf16_tflops_sustained"],
                    "traffic": traffic, "traffic_source": traffic_src, "peak_kind": peak_kind + " (sustained)",
                    "hbm_gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"],
                    "frac_whole_call": attn_flops / (t_call * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]}
        am_traffic, am_src = ncu_traffic("argmax", args.workload)
        kernels = {
            "verify_attn": {"kernel_ms": t_attn_kernel, "call_ms": t_call, "call_ms_in_step": t_attn_in_step,
                            "algorithmic_bytes": attn_bytes, "gbs": gbs, "algorithmic_flops": attn_flops, "tflops": tfs,
                            "binding_bound": bound, "binding_frac": max(t_hbm, t_tc) / (t_attn_kernel * 1e-3),
                            "note": "kernel_ms: attention kernel alone (events inside the call); call_ms: the headline, "
                                    "one call of back-to-back calls (preparation + attention + combine, launches overlapping)"},
            "accept": {"argmax_kernel_ms": t_argmax_kernel, "walk_call_ms": t_walk, "accept_commit_call_ms": t_accept,
                       "algorithmic_bytes": w.logits_bytes(), "gbs": w.logits_bytes() / (t_argmax_kernel * 1e-3) / 1e9,
                       "hbm_frac": w.logits_bytes() / (t_argmax_kernel * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       "traffic": am_traffic, "traffic_source": am_src,
                       "note": "argmax_kernel_ms / gbs: the target argmax over the logits alone; walk_call_ms: reader_accept "
                               "from given target ids; accept_commit_call_ms: reader_accept_commit from logits inside the step "
                               "(argmax, then walk and commit in one launch)"},
            "kv_commit": {"call_ms": t_commit, "note": "reader_kv_commit alone, one layer"},
        }
        kernels.update(extras.get("kernels", {}))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": t_call, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": workload_config(w, args.workload),
            "timed": {"blocks": n_blocks, "steps_per_block": K, "timed_region_ms": sum(block_ms), "block_ms_median": ms_block,
                      "block_ms_min": min(block_ms), "block_ms_max": max(block_ms),
                      "note": "a step = one reader_verify_attn call; blocks of `steps` calls repeated until about a second "
                              "is timed, the median block is reported"},
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "blocks": ne,
                    "ms_per_step": ms_e2e_block / K},
            # C1 and C2 take the single-launch form of the attention kernel (unless a kernel was forced)
            "gpu_launches": (1 if (args.workload in ("c1", "c2") and args.kernel in (0, 3)) else LAUNCHES_PER_ATTN_CALL) * K * n_blocks,
            "clocks": clocks, "roofline": roof,
            "whole_step": {"ms_per_step": t_step, "tokens_per_s": tokens / (t_step * 1e-3), "launches_per_step": LAUNCHES_PER_STEP,
                           "steps": Ks, "note": "reader_verify_attn (masks encoded inside) + reader_accept_commit from logits, "
                                                "back to back; reported beside the metric, not folded into it"},
            "kernels": kernels,
        }
        for k in ("cuda_graph_replay", "model_step"):
            if k in extras:
                line[k] = extras[k]
        if table is not None:
            line["workloads"] = table
        if long_prefix is not None:
            line["shared_prefix_larger_than_l2"] = long_prefix
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    rd.close()


def run_extras(args, rd, w, d, dev, rank, step, seq_lens0, out, status, ws, tgt, acc_out, slots, cstat, barrier, mk):
    """What surrounds the metric: the step as a CUDA graph, a 32-layer model step, batched commits, the
    sampling policy's kernel and Algorithm 4 on a padded cache.  None of it enters `value`."""
    import torch
    from paper_2508_09072_b200 import binding
    B, T = w.batch, w.n_nodes
    res = {"kernels": {}}

    # ---- the whole step captured once in a CUDA graph and replayed (no host work per step)
    try:
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                step()
        torch.cuda.synchronize()
        for _ in range(5):
            graph.replay()
        Kg = 200
        barrier()
        g0, g1 = mk(), mk()
        g0.record()
        for _ in range(Kg):
            graph.replay()
        g1.record()
        barrier()
        t_graph = g0.elapsed_time(g1) / Kg
        res["cuda_graph_replay"] = {"ms_per_step": t_graph, "tokens_per_s": B * T / (t_graph * 1e-3), "what": "the whole step"}
    except Exception as exc:                                  # reported, never hidden
        res["cuda_graph_replay"] = f"capture failed: {exc}"

    # ---- a 32-layer model's commits: layer by layer against one batched launch
    n_layers = 32
    layer_caches = [d.cache] * n_layers
    lk, lv = [d.k_tree] * n_layers, [d.v_tree] * n_layers

    def commits_one_by_one():
        d.cache.seq_lens.copy_(seq_lens0)
        for i in range(n_layers):
            rd.kv_commit(d.cache, d.k_tree, d.v_tree, acc_out[0], acc_out[1], update_seq_lens=(i == n_layers - 1),
                         slots=slots, status=cstat)

    def commits_batched():
        d.cache.seq_lens.copy_(seq_lens0)
        rd.kv_commit_layers(layer_caches, lk, lv, acc_out[0], acc_out[1], slots=slots, status=cstat)

    t_layers = {}
    for label, fn in (("one_by_one", commits_one_by_one), ("batched", commits_batched)):
        fn()
        c0, c1 = mk(), mk()
        c0.record()
        for _ in range(20):
            fn()
        c1.record()
        barrier()
        t_layers[label] = c0.elapsed_time(c1) / 20
    res["kernels"]["kv_commit_32_layers"] = {"call_ms": t_layers, "note": "the accepted rows committed into 32 layers: 32 calls of "
                                             "reader_kv_commit against one reader_kv_commit_layers"}

    # ---- a whole model's verification step: every layer's attention over that layer's own cache (device
    # copies of the pool, one block table for the model), one acceptance, one commit into all layers;
    # issued call by call, then captured once in a CUDA graph and replayed
    try:
        pool_bytes = 2 * d.cache.k_pool.numel() * d.cache.k_pool.element_size()
        Lm = max(2, min(n_layers, int(40e9 // max(pool_bytes, 1))))
        m_caches = [d.cache] + [binding.KvCache(d.cache.k_pool.clone(), d.cache.v_pool.clone(), d.cache.page_table,
                                                d.cache.seq_lens, d.cache.shared_prefix_len) for _ in range(Lm - 1)]

        def model_step():
            d.cache.seq_lens.copy_(seq_lens0)
            rd.verify_prepare(m_caches[0], d.parent, w.n_q_heads, status=status, workspace=ws)   # once for all layers
            for c in m_caches:
                rd.verify_attn_prepared(d.q, d.k_tree, d.v_tree, c, d.parent, w.scale, ws, out=out)
            rd.accept(d.parent, d.node_tokens, w.max_path, logits=d.logits, target_ids=tgt, workspace=ws, outs=acc_out)
            rd.kv_commit_layers(m_caches, lk[:Lm], lv[:Lm], acc_out[0], acc_out[1], slots=slots, status=cstat)

        for _ in range(2):
            model_step()
        m0, m1 = mk(), mk()
        m0.record()
        for _ in range(10):
            model_step()
        m1.record()
        barrier()
        t_model_eager = m0.elapsed_time(m1) / 10
        side2 = torch.cuda.Stream()
        with torch.cuda.stream(side2):
            model_step()
            torch.cuda.synchronize()
            mgraph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(mgraph, stream=side2):
                model_step()
        torch.cuda.synchronize()
        for _ in range(3):
            mgraph.replay()
        barrier()
        m2, m3 = mk(), mk()
        m2.record()
        for _ in range(20):
            mgraph.replay()
        m3.record()
        barrier()
        t_model_graph = m2.elapsed_time(m3) / 20
        assert int(status.max().item()) == 0 and int(cstat.max().item()) == 0
        kv_bytes = Lm * w.attn_algorithmic_bytes() + w.logits_bytes()
        best = min(t_model_eager, t_model_graph)
        res["model_step"] = {"layers": Lm, "ms_per_step": {"call_by_call": t_model_eager, "cuda_graph": t_model_graph},
                             "ms_per_layer": (best - 0.0) / Lm, "tokens_per_s": B * T / (best * 1e-3), "algorithmic_bytes": kv_bytes,
                             "gbs": kv_bytes / (best * 1e-3) / 1e9,
                             "note": "checks and work partition once, every layer's verify attention on its own cache, one "
                                     "acceptance, one commit into all layers; reported beside the metric"}
        del m_caches, mgraph
        torch.cuda.empty_cache()
    except Exception as exc:                                  # reported, never hidden
        res["model_step"] = f"failed: {exc}"

    # ---- the sampling policy's target kernel (an alternative to the argmax; not part of the step)
    uni = torch.rand((B, T), dtype=torch.float32, device=dev)
    tgt_s = torch.empty((B, T), dtype=torch.int32, device=dev)

    def time_sample(n, **kw):
        for _ in range(2):
            rd.sample_targets(d.parent, d.logits, uni, 0.8, target_ids=tgt_s, **kw)
        a, b = mk(), mk()
        a.record()
        for _ in range(n):
            rd.sample_targets(d.parent, d.logits, uni, 0.8, target_ids=tgt_s, **kw)
        b.record()
        barrier()
        return a.elapsed_time(b) / n

    t_sample = time_sample(20)
    res["kernels"]["sample_targets"] = {
        "call_ms": t_sample, "algorithmic_bytes": w.logits_bytes(), "gbs": w.logits_bytes() / (t_sample * 1e-3) / 1e9,
        "variants_call_ms": {"top_k_50": time_sample(10, top_k=50), "top_p_0.9": time_sample(5, top_p=0.9),
                             "top_k_50_top_p_0.9": time_sample(5, top_k=50, top_p=0.9)},
        "note": "sampling policy (Appendix C, temperature 0.8); replaces the argmax when used; flat synthetic logits, so "
                "the nucleus for 0.9 holds tens of thousands of tokens"}

    # ---- the paper's own cache maintenance (Algorithm 4) on a padded batch cache of the same size class
    capR, gen = 4096, torch.Generator(device=dev)
    gen.manual_seed(1234 + rank)
    kR = torch.randn((B, w.n_kv_heads, capR, w.head_dim), device=dev, generator=gen).to(torch.bfloat16)
    vR = kR.clone()
    maskR0 = (torch.rand((B, capR), device=dev, generator=gen) < 0.85).to(torch.uint8)
    maskR0[:, : capR // 2] = 1                               # the first half is already compact
    maskR, lenR = maskR0.clone(), torch.empty(B, dtype=torch.int32, device=dev)
    rd.kv_rearrange(kR, vR, maskR, lenR)
    r_times = []
    for _ in range(5):
        maskR.copy_(maskR0)                                  # same holes again (the data has moved; the cost is the same)
        r0, r1 = mk(), mk()
        r0.record(); rd.kv_rearrange(kR, vR, maskR, lenR); r1.record()
        torch.cuda.synchronize()
        r_times.append(r0.elapsed_time(r1))
    t_rearr = median(r_times)
    rearr_bytes = 2 * 2 * (B * w.n_kv_heads * (capR - capR // 2) * w.head_dim * 2)   # K and V, read + write of the moving half
    res["kernels"]["kv_rearrange"] = {"call_ms": t_rearr, "moved_bytes": rearr_bytes, "gbs": rearr_bytes / (t_rearr * 1e-3) / 1e9,
                                      "note": "Algorithm 4 on a padded batch cache [B][Hkv][4096][D], 85 % valid behind a compact "
                                              "first half"}
    del kR, vR
    return res


# ------------------------------------------------------------------------------------------------
# tree-size sweep: T_V(T), the verification-attention time as a function of the draft-tree size
# (Sec. 3.2: reads grow with s + gamma, FLOPs with gamma (s + gamma); Theorem 1 needs T_V(T))
# ------------------------------------------------------------------------------------------------
def run_sweep(args):
    import numpy as np
    import torch
    from paper_2508_09072_b200 import binding, workloads as W
    torch.cuda.set_device(0)
    rd = binding.Reader(0)
    flush = make_flush()
    peaks, _ = load_peaks()
    rows = []
    for B in (1, 8, 32):
        for T in (8, 16, 32, 64, 128):
            rng = np.random.default_rng(77 + B)
            lens = rng.integers(1024, 4097, size=B)
            w = W.build_workload(f"sweep-b{B}-t{T}", 9000 + 131 * B + T, lens, T, 32, 8, 128,
                                 lambda r: W.capped_recursive_tree(r, T, 12, 4), max_path=12, vocab=16,
                                 shuffle_pages=True, with_logits=False)
            d = binding.to_device(w, with_logits=False)
            anc, _, _ = rd.tree_encode(d.parent)
            out = torch.empty_like(d.q)
            st = torch.empty(B, dtype=torch.int32, device="cuda")
            ws = rd.workspace(B, T, 32, 8, 128)
            call = lambda: rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, anc_mask=anc, out=out,
                                          status=st, workspace=ws)
            for _ in range(3):
                call()
            ts = []
            for _ in range(args.sweep_iters):
                flush()                                        # cold L2: the small cases fit in it
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); call(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            ts.sort()
            us = ts[len(ts) // 2] * 1e3
            t_hbm = w.attn_algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9) * 1e6
            t_tc = w.attn_algorithmic_flops() / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6
            rows.append({"batch": B, "tree_nodes": T, "committed_tokens": int(lens.sum()), "call_us": us,
                         "tokens_per_s": B * T / (us * 1e-6), "t_hbm_us": t_hbm, "t_tensor_us": t_tc,
                         "bound": "hbm" if t_hbm >= t_tc else "tensor"})
    print(json.dumps({"sweep": "verify-attention call time vs draft-tree size (cold L2, median)", "rows": rows}))
    rd.close()


# ------------------------------------------------------------------------------------------------
# verify attention alone on all five workloads (cold L2): the numbers behind the roofline table
# ------------------------------------------------------------------------------------------------
def make_flush(dev="cuda"):
    """A read pass over 512 MB (four times the L2): see run_ours."""
    import torch
    buf = torch.zeros((512 << 20) // 4, dtype=torch.int32, device=dev)
    sink = torch.zeros((), dtype=torch.int64, device=dev)
    return lambda: torch.sum(buf, dim=(0,), out=sink)


def run_attn_table(args):
    import torch
    from paper_2508_09072_b200 import binding, workloads as W
    torch.cuda.set_device(0)
    rd = binding.Reader(0)
    if args.kernel:
        rd.set_attn_kernel(args.kernel)
    flush = make_flush()
    peaks, peak_kind = load_peaks()
    rows = []
    for name in W.WORKLOADS:
        case = AttnCase(rd, W.make(name, with_logits=False), "cuda:0")
        rows.append(attn_row(case, flush, peaks, args.table_iters, 30.0))
        del case
        torch.cuda.empty_cache()
    print(json.dumps({"table": "verify attention per workload, L2 flushed (read pass) before every call, median", "peaks": peaks,
                      "peak_kind": peak_kind, "rows": rows}))
    rd.close()


# ------------------------------------------------------------------------------------------------
# a shared prefix that does not fit the L2: the equal-range partition against the aligned one
# ------------------------------------------------------------------------------------------------
def long_prefix_rows(rd, dev, peaks, iters, partitions=(1, 2)):
    """16 sequences over one 32 768-token prefix (134 MB of K and V) plus private suffixes: attention kernel
    time under both work partitions.  How often the prefix comes from HBM is in the ncu summary under
    profiles/ (counters need the profiler); here only times."""
    import torch
    from paper_2508_09072_b200 import workloads as W
    case = AttnCase(rd, W.make_long_shared_prefix(), dev)
    w = case.w
    mk = lambda: torch.cuda.Event(enable_timing=True)
    rows = []
    for part in partitions:
        rd.set_partition(part)
        for _ in range(3):
            case.call()
        ts = []
        for _ in range(iters):
            c, e = mk(), mk()
            c.record(); e.record()
            rd.set_timing_events(c, e)
            case.call()
            torch.cuda.synchronize()
            ts.append(c.elapsed_time(e))
        rd.set_timing_events(None, None)
        assert int(case.status.max().item()) == 0
        k = median(ts) * 1e-3
        by, fl = w.attn_algorithmic_bytes(), w.attn_algorithmic_flops()
        rows.append({"partition": {1: "equal ranges", 2: "aligned (the automatic choice at this size)"}[part], "kernel_us": k * 1e6,
                     "algorithmic_bytes": by, "gbs": by / k / 1e9, "algorithmic_flops": fl, "tflops": fl / k / 1e12,
                     "tensor_frac": fl / k / 1e12 / peaks["bf16_tflops_sustained"]})
    rd.set_partition(0)
    return {"workload": "16 sequences sharing a 32768-token prefix (134 MB of K+V) + private suffixes of 256..1024, 32-node trees",
            "l2": "no flush: every call streams more K/V than the 126 MB L2 holds", "rows": rows}


def run_long_prefix(args):
    import torch
    from paper_2508_09072_b200 import binding
    torch.cuda.set_device(0)
    rd = binding.Reader(0)
    peaks, _ = load_peaks()
    parts = (1, 2) if args.partition == 0 else (args.partition,)
    print(json.dumps(long_prefix_rows(rd, "cuda:0", peaks, args.table_iters, parts)))
    rd.close()


# ------------------------------------------------------------------------------------------------
# the paper's padded batch cache against the paged cache over a run of decoding steps (Sec. 4.3)
# ------------------------------------------------------------------------------------------------
def run_cache_sim(args):
    """Many verification steps with drawn accepted spans (geometric lengths, now and then a long span from
    the statistical search): attention + cache maintenance per step, for the paged cache and for the padded
    batch cache rearranged every N steps (Algorithm 4), N = 10, 25, 50 and never."""
    import numpy as np
    import torch
    from paper_2508_09072_b200 import binding, workloads as W
    torch.cuda.set_device(0)
    rd = binding.Reader(0)
    B, T, Hq, Hkv, D = 32, 32, 32, 8, 128
    prompt, steps, chain, accept_rate, p_long = 1024, args.sim_steps, 16, 0.7, 0.03
    max_path = chain
    cap = -(-(prompt + steps * max_path) // 64) * 64
    w = W.build_workload("cache-sim", 4242, [prompt] * B, T, Hq, Hkv, D,
                         lambda r: W.widened_tree(r, T, chain, 6, 4), max_path=max_path, vocab=16, shuffle_pages=True,
                         with_logits=False, room=steps * max_path)
    rng = np.random.default_rng(4243)
    spans = [W.accepted_spans(rng, B, T, max_path, w.parent, accept_rate, p_long) for _ in range(steps)]
    paths = torch.from_numpy(np.stack([s[0] for s in spans])).cuda()
    n_accs = torch.from_numpy(np.stack([s[1] for s in spans])).cuda()
    grown = int(sum(int(s[1].max()) for s in spans))
    real = np.stack([s[1] for s in spans]).sum(axis=0)

    d = binding.to_device(w, with_logits=False)
    anc, _, _ = rd.tree_encode(d.parent)
    pc = W.padded_cache_of(w, seed=1, slack=0, capacity=cap)
    cache = binding.padded_to_device(pc)
    valid0, lens0 = cache.valid.clone(), d.cache.seq_lens.clone()
    out_paged, out_padded = torch.empty_like(d.q), torch.empty_like(d.q)
    st = torch.empty(B, dtype=torch.int32, device="cuda")
    slots = torch.empty((B, max_path), dtype=torch.int32, device="cuda")
    lengths = torch.empty(B, dtype=torch.int32, device="cuda")
    ws = torch.empty(int(rd.lib.reader_padded_workspace_bytes(rd._h, B, T, Hq, Hkv, D, cap)), dtype=torch.uint8, device="cuda")
    bad = torch.zeros(1, dtype=torch.int32, device="cuda")
    mk = lambda: torch.cuda.Event(enable_timing=True)

    def run_paged():
        d.cache.seq_lens.copy_(lens0)
        a, b = mk(), mk()
        a.record()
        for s in range(steps):
            rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, anc_mask=anc, out=out_paged, status=st, workspace=ws)
            bad.add_(st.max())
            rd.kv_commit(d.cache, d.k_tree, d.v_tree, paths[s], n_accs[s], slots=slots, status=st)
            bad.add_(st.max())
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    def run_padded(every):
        cache.valid.copy_(valid0)
        cache.extent.fill_(prompt)
        peak = torch.zeros(1, dtype=torch.int32, device="cuda")
        a, b = mk(), mk()
        a.record()
        for s in range(steps):
            rd.verify_attn_padded(d.q, d.k_tree, d.v_tree, cache, d.parent, w.scale, anc_mask=anc, out=out_padded, status=st,
                                  workspace=ws)
            bad.add_(st.max())
            rd.padded_append(cache, d.k_tree, d.v_tree, paths[s], n_accs[s], status=st)
            bad.add_(st.max())
            torch.maximum(peak, cache.extent, out=peak)
            if every and s % every == every - 1:
                rd.padded_rearrange(cache, lengths)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b), int(peak.item()), int(cache.extent.item())

    # the same attention call on the two layouts while they still hold the same compact content
    flush = make_flush()

    def call_us(call):
        for _ in range(3):
            call()
        ts = []
        for _ in range(args.sweep_iters):
            flush()
            a, b = mk(), mk()
            a.record(); call(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return sorted(ts)[len(ts) // 2] * 1e3
    first_call = {
        "paged": call_us(lambda: rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, anc_mask=anc,
                                                out=out_paged, status=st, workspace=ws)),
        "padded": call_us(lambda: rd.verify_attn_padded(d.q, d.k_tree, d.v_tree, cache, d.parent, w.scale, anc_mask=anc,
                                                        out=out_padded, status=st, workspace=ws))}
    del flush

    run_paged()                                               # warm-up: descriptors, caches, clocks
    t_paged = sorted(run_paged() for _ in range(3))[1]
    assert d.cache.seq_lens.cpu().numpy().tolist() == (prompt + real).tolist()
    rows = []
    for every in (10, 25, 50, 0):
        run_padded(every)
        res = sorted(run_padded(every) for _ in range(3))[1]
        assert cache.valid.sum(dim=1).cpu().numpy().tolist() == (prompt + real).tolist()
        rows.append({"rearrange_every": every or "never", "ms_total": res[0], "us_per_step": res[0] / steps * 1e3,
                     "vs_paged": res[0] / t_paged, "peak_extent": res[1], "final_extent": res[2]})
    # the two designs hold the same entries: one more verification on the final caches must agree
    rd.verify_attn(d.q, d.k_tree, d.v_tree, d.cache, d.parent, w.scale, anc_mask=anc, out=out_paged, status=st, workspace=ws)
    rd.verify_attn_padded(d.q, d.k_tree, d.v_tree, cache, d.parent, w.scale, anc_mask=anc, out=out_padded, status=st, workspace=ws)
    torch.cuda.synchronize()
    diff = float((out_paged.float() - out_padded.float()).abs().max().item())
    assert int(bad.item()) == 0 and diff <= 2e-2, (int(bad.item()), diff)
    by_n = {r["rearrange_every"]: r["ms_total"] for r in rows}
    print(json.dumps({
        "cache_sim": "verify attention + cache maintenance per step: paged cache against the padded batch cache of Sec. 4.3",
        "config": {"batch": B, "tree_nodes": T, "n_q_heads": Hq, "n_kv_heads": Hkv, "head_dim": D, "prompt_len": prompt,
                   "steps": steps, "accept_rate": accept_rate, "p_long_span": p_long, "long_span": chain,
                   "p_some_sample_long": 1 - (1 - p_long) ** B, "capacity": cap,
                   "l2": "no flush: each step reads more KV than the 126 MB L2 holds"},
        "accepted_per_sample_per_step": float(real.mean() / steps), "common_growth_per_step": grown / steps,
        "attention_call_us_on_the_compact_initial_cache": first_call,
        "paged": {"ms_total": t_paged, "us_per_step": t_paged / steps * 1e3},
        "padded": rows,
        "rearrangement_gain_n25_vs_never": 1 - by_n[25] / by_n["never"],
        "max_abs_diff_final_outputs": diff}))
    rd.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--kernel", type=int, default=0, help="attention kernel: 0 auto, 1 CUDA-core, 2 tensor-core")
    ap.add_argument("--min-timed-ms", type=float, default=1000.0, help="blocks of --steps calls are repeated until about this much is timed")
    ap.add_argument("--table-iters", type=int, default=15, help="calls per measurement in the five-workload table")
    ap.add_argument("--no-table", action="store_true", help="skip the five-workload table")
    ap.add_argument("--quick", action="store_true", help="skip what surrounds the metric (graph, model step, sampling, rearrangement)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep-tree", action="store_true", help="measure the attention call for several tree sizes instead")
    ap.add_argument("--sweep-iters", type=int, default=15)
    ap.add_argument("--attn-table", action="store_true", help="verify attention alone on C1..C5 instead")
    ap.add_argument("--long-prefix", action="store_true", help="a shared prefix larger than L2 under both work partitions instead")
    ap.add_argument("--partition", type=int, default=0, help="with --long-prefix: 1 equal ranges only, 2 aligned only")
    ap.add_argument("--cache-sim", action="store_true", help="paged cache against the paper's padded batch cache over many steps instead")
    ap.add_argument("--sim-steps", type=int, default=200)
    args = ap.parse_args()
    if args.attn_table:
        run_attn_table(args)
    elif args.cache_sim:
        run_cache_sim(args)
    elif args.long_prefix:
        run_long_prefix(args)
    elif args.sweep_tree:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
