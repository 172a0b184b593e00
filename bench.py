#!/usr/bin/env python
"""Benchmark of the FSM-indexed guided-generation hot path on B200.

One *step* is one pass of the whole path over one batch of synthetic input:
``fsm_index_build`` for the Llama-3-shaped workload (1,001 states x 128,256
tokens, int32 next-state table) followed by one ``guided_mask_step`` over
B = 256 bf16 logits rows of that vocabulary, in place.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line.  ``value`` is (state, token) walks per second of the index
build (Q*N per build, all ranks, divided by the build's device time inside the
step); ``mask_step_us`` is the masked-logit step (``sample_step_us`` the same step with the
categorical draw at temperature 0.1 instead of the argmax); ``ms_per_step`` is the
whole step.  With N > 1 (torchrun) every rank runs the same-shaped workload on its own
GPU with its own automaton seed: the path shards over independent problems and
has no data-path collective (weak scaling).

``--shard states`` measures the other split instead: ONE workload-4 index (20,001 states
x 152,064 tokens) divided over the ranks by state slabs, every rank building its slab with
``fsm_index_build_rows`` and the slabs meeting in an NCCL all-gather (strong scaling).

``--impl reference`` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "index build (state,token) walks/s; masked-logit step us at B=256, N=128k"
UNIT = "walks/s"
B_ROWS = 256
# DRAM bytes (read + write) per launch come from the ncu summaries under profiles/: each
# names the kernel source it was captured from with that file's SHA-256, and a summary whose
# source has changed since gives no figure (see ncu_traffic()).
PROFILES = {"walk_rows": "walk_rows_config3.md", "mask_step": "mask_step_config5.md"}
# kernels of this library per timed step: prepare_fused, walk_rows, mask_step
LAUNCHES_PER_STEP = 3
RING = 8


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def ncu_traffic(kind: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of the first captured launch in the
    profile summary of `kind`, or None when there is no summary or the kernel's source file
    is no longer the one the capture was taken from."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", PROFILES[kind])
    try:
        text = open(path).read()
    except OSError:
        return None
    m = re.search(r"source:\s*(\S+)\s+sha256=([0-9a-f]+)", text)
    if not m:
        return None
    try:
        digest = hashlib.sha256(open(os.path.join(ROOT, m.group(1)), "rb").read()).hexdigest()
    except OSError:
        return None
    if not digest.startswith(m.group(2)):
        return None
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    total = 0.0
    for name in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        row = re.search(r"^\|\s*" + re.escape(name) + r"\s*\|\s*(\w+)\s*\|\s*([0-9.eE+-]+)", text, re.M)
        if not row or row.group(1) not in scale:
            return None
        total += float(row.group(2)) * scale[row.group(1)]
    return total


def lookups_per_walk(w, threads, n_states=48):
    """Table look-ups an early-exit walk makes per (state, token) pair, counted by the oracle
    on a sample of the states (spread over the automaton)."""
    from oracle import fsm_oracle
    d = w.dfa
    total, pairs = 0, 0
    step = max(1, d.Q // n_states)
    for q in range(0, d.Q, step):
        _, _, n = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                         w.eos_id, q_begin=q, q_end=q + 1, want_next=False,
                                         threads=threads)
        total += int(n)
        pairs += w.N
    return total / pairs


def workload(rank: int):
    """Workload 3 (index) + workload 5 (decode batch); rank r > 0 draws its own
    automaton of the same shape."""
    from fsm_inputs import make_config, random_class_dfa, start_states
    w = make_config(5)
    if rank > 0:
        w.dfa, _ = random_class_dfa(w.seed + 5000 + rank, 1000, 64, 12, 0.10)
    return w, start_states(w)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_index_rate(w, threads, budget_s):
    """Times the oracle's index build on a bounded sample of states."""
    from oracle import fsm_oracle
    d = w.dfa
    t0 = time.perf_counter()
    fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                           q_begin=0, q_end=min(16, d.Q), threads=threads)
    per_state = max((time.perf_counter() - t0) / min(16, d.Q), 1e-6)
    n_states = int(max(1, min(d.Q, budget_s / per_state)))
    t0 = time.perf_counter()
    fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                           q_begin=0, q_end=n_states, threads=threads)
    dt = time.perf_counter() - t0
    return n_states * w.N / dt, n_states, dt


def cpu_baseline(w, starts):
    from fsm_inputs import f32_to_bf16_bits, step_logits_numpy
    from oracle import fsm_oracle
    threads = len(os.sched_getaffinity(0))
    rate, n_states, dt = oracle_index_rate(w, threads, budget_s=8.0)
    d = w.dfa
    # the whole workload fits the budget on a many-core host: repeat it for about 10 s of work
    reps_index, spent, best = 1, dt, dt
    while spent < 10.0 and reps_index < 200:
        t0 = time.perf_counter()
        fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                               q_begin=0, q_end=n_states, threads=threads)
        t = time.perf_counter() - t0
        best, spent, reps_index = min(best, t), spent + t, reps_index + 1
    rate, dt = n_states * w.N / best, best
    mask, nxt, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                          w.eos_id, threads=threads)
    logits = f32_to_bf16_bits(step_logits_numpy(w, 0))
    reps, t_mask = 3, []
    for _ in range(reps):
        st, fin = starts.copy(), np.zeros(w.B, np.uint8)
        t0 = time.perf_counter()
        fsm_oracle.mask_step(logits, st, fin, mask, nxt, d.dead, w.eos_id, threads=threads)
        t_mask.append(time.perf_counter() - t0)
    return {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"index build of states 0..{n_states - 1} of {d.Q} x all {w.N} tokens "
                      f"(best of {reps_index} runs, {dt:.3f} s each, OpenMP over states); "
                      f"mask step: {reps} full B=256 steps",
            "mask_step_us": float(np.median(t_mask) * 1e6)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w, starts = workload(0)
    threads = len(os.sched_getaffinity(0))
    total = max(1, args.steps + args.warmup)
    budget = min(20.0, 150.0 / total)              # seconds of oracle work per step
    from fsm_inputs import f32_to_bf16_bits, step_logits_numpy
    from oracle import fsm_oracle
    d = w.dfa
    rate, n_states, _ = oracle_index_rate(w, threads, budget * 0.8)
    rows = int(max(1, min(w.B, round(w.B * budget * 0.2 / 0.1))))   # ~0.1 s per full step on 8 cores
    mask, nxt, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                          w.eos_id, threads=threads)
    logits = f32_to_bf16_bits(step_logits_numpy(w, 0))[:rows].copy()
    t_build, t_mask = [], []
    for it in range(total):
        t0 = time.perf_counter()
        fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                               q_begin=0, q_end=n_states, threads=threads)
        t1 = time.perf_counter()
        st, fin = starts[:rows].copy(), np.zeros(rows, np.uint8)
        fsm_oracle.mask_step(logits, st, fin, mask, nxt, d.dead, w.eos_id, threads=threads)
        t2 = time.perf_counter()
        if it >= args.warmup:
            t_build.append(t1 - t0)
            t_mask.append(t2 - t1)
    value = n_states * w.N / float(np.mean(t_build))
    mask_us = float(np.mean(t_mask)) * 1e6 * (w.B / rows)
    sample = (f"per step: oracle index build of {n_states} of {d.Q} states x {w.N} tokens, and "
              f"the oracle mask step on {rows} of {w.B} rows (scaled to {w.B})")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": float(np.mean(t_build) + np.mean(t_mask)) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic", "mask_step_us": mask_us,
        "config": config_dict(w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def config_dict(w, n_gpus):
    return {"workload": "index build: Llama-3-shaped vocab N=128256, random DFA Q=1001 (12 live "
                        "byte classes/state), int32 next-state + packed bitmask; then one mask "
                        "step: B=256 bf16 logits [256x128256], in place",
            "Q": w.Q, "N": w.N, "B": w.B, "state_dtype": "int32", "logits_dtype": "bf16",
            "parallelism": f"independent problems x{n_gpus}, no collective",
            "l2": f"inputs larger than L2, no explicit flush: per step 529 MB of index output is "
                  f"written between mask steps, and the logits come from a ring of {RING} x 65.7 MB "
                  f"buffers (the 126 MB L2 holds less than two)"}


# --------------------------------------------------------------------------- GPU arm
def run_ours(args):
    import torch
    import paper_2307_09702_b200 as fg
    from paper_2307_09702_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if fg.fsm_device_check() != 0:
        raise SystemExit("bench.py needs a compute-capability 10.x device")
    dev = torch.device("cuda", local)
    fg.fsm_debug_set(binding.FSM_TUNE_WALK_ALGO, args.walk_algo)
    w, starts = workload(rank)
    d = w.dfa
    idx = fg.GuidedIndex(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                         fg.FSM_STATE_I32, True, device=dev)
    sigma = w.logits_sigma
    g = torch.Generator(device=dev).manual_seed(w.seed)
    ring = [(torch.randn((w.B, w.N), generator=g, device=dev) * sigma).to(torch.bfloat16)
            for _ in range(RING)]
    st0 = torch.from_numpy(starts).to(dev)
    fin0 = torch.zeros(w.B, dtype=torch.uint8, device=dev)
    st, fin = st0.clone(), fin0.clone()
    tok = torch.zeros(w.B, dtype=torch.int32, device=dev)

    def step(i, ev=None):
        st.copy_(st0)
        fin.copy_(fin0)
        if ev:
            ev[0].record()
        idx.build()
        if ev:
            ev[1].record()
        idx.step(ring[i % RING], st, fin, tok)
        if ev:
            ev[2].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    assert int(idx.status.item()) == 0, "data-fault flag raised during warm-up"

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fg.fsm_debug_set(binding.FSM_PROFILE_WALK, 1)
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    t_begin.record()
    for i in range(args.steps):
        step(i, events[i])
    t_end.record()
    barrier()
    clocks = sampler.stop()
    fg.fsm_debug_set(binding.FSM_PROFILE_WALK, 0)
    walk_ms = fg.fsm_profile_read()[: args.steps]
    total_ms = t_begin.elapsed_time(t_end)

    # ---- the mask step alone, back to back over the logits ring (inputs larger than L2),
    # as a decode loop runs it: states advance from step to step
    m_begin, m_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    mask_loop_steps = max(args.steps, 200)
    st.copy_(st0)
    fin.copy_(fin0)
    for i in range(args.warmup):
        idx.step(ring[i % RING], st, fin, tok)
    st.copy_(st0)
    fin.copy_(fin0)
    barrier()
    m_begin.record()
    for i in range(mask_loop_steps):
        idx.step(ring[i % RING], st, fin, tok)
    m_end.record()
    barrier()
    mask_loop_ms = m_begin.elapsed_time(m_end) / mask_loop_steps
    rows_live_end = int((fin == 0).sum().item())
    # ---- the same loop with the categorical draw (temperature 0.1, as in the paper's runs)
    st.copy_(st0)
    fin.copy_(fin0)
    for i in range(args.warmup):
        idx.sample(ring[i % RING], st, fin, tok, 10.0, w.seed, i)
    st.copy_(st0)
    fin.copy_(fin0)
    barrier()
    m_begin.record()
    for i in range(mask_loop_steps):
        idx.sample(ring[i % RING], st, fin, tok, 10.0, w.seed, 1000 + i)
    m_end.record()
    barrier()
    sample_ms = m_begin.elapsed_time(m_end) / mask_loop_steps
    build_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in events]))
    mask_in_step_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in events]))
    mask_ms = mask_loop_ms
    walk_ms_mean = float(np.mean(walk_ms)) if walk_ms else float("nan")

    # ---- the other output modes of the index build (not part of the timed step)
    def time_build(state_dtype, want_next, n=20, wl=None):
        wl = wl or w
        dd = wl.dfa
        other = fg.GuidedIndex(dd.trans, dd.accept, wl.vocab_bytes, wl.vocab_offsets, dd.dead, wl.eos_id,
                               state_dtype, want_next, device=dev)
        for _ in range(3):
            other.build()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            other.build()
        b.record()
        torch.cuda.synchronize()
        assert int(other.status.item()) == 0
        return a.elapsed_time(b) / n

    u16_ms = time_build(fg.FSM_STATE_U16, True)
    maskonly_ms = time_build(fg.FSM_STATE_I32, False)

    def time_csr(n=20):
        """The index as compressed rows (allowed token lists with end states)."""
        cap = int(0.08 * w.Q * w.N)
        off = torch.empty(w.Q + 1, dtype=torch.int64, device=dev)
        ctok = torch.empty(cap, dtype=torch.int32, device=dev)
        cnext = torch.empty(cap, dtype=torch.int32, device=dev)

        def run():
            rc = fg.fsm_index_build_csr(idx.trans, idx.accept, idx.vocab_bytes, idx.vocab_offsets,
                                        idx.vocab_nbytes, w.Q, w.N, d.dead, w.eos_id, idx.allowed_mask,
                                        off, ctok, cnext, cap, idx.workspace, idx.workspace_bytes,
                                        idx.status)
            assert rc == 0
        for _ in range(3):
            run()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            run()
        b.record()
        torch.cuda.synchronize()
        assert int(idx.status.item()) == 0, "compressed-row capacity too small"
        return a.elapsed_time(b) / n, int(off[-1].item())

    csr_ms, csr_nnz = time_csr()
    idx.build()    # the dense index again, for the end-to-end loop below

    def time_alias(n=20):
        """Merging of identical rows of the built int32 index (reads every row once)."""
        alias = torch.empty(w.Q, dtype=torch.int32, device=dev)
        uniq = torch.zeros(1, dtype=torch.int32, device=dev)
        wsb = fg.fsm_row_alias_workspace_bytes(w.Q)
        ws = torch.empty(wsb, dtype=torch.uint8, device=dev)

        def run():
            rc = fg.fsm_index_row_alias(idx.allowed_mask, idx.next_state, fg.FSM_STATE_I32, w.Q, w.N, alias,
                                        uniq, ws, wsb, idx.status)
            assert rc == 0
        for _ in range(3):
            run()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(n):
            run()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / n, int(uniq.item())

    alias_ms, alias_unique = time_alias()

    # ---- end to end: host buffers in, host results out, through the same calls
    host = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in {
        "trans": d.trans, "accept": d.accept, "vb": w.vocab_bytes, "vo": w.vocab_offsets,
        "states": starts}.items()}
    host_logits = ring[0].cpu().pin_memory()
    host_fin = torch.zeros(w.B, dtype=torch.uint8).pin_memory()
    out_tok = torch.empty(w.B, dtype=torch.int32).pin_memory()
    out_st = torch.empty(w.B, dtype=torch.int32).pin_memory()
    out_fin = torch.empty(w.B, dtype=torch.uint8).pin_memory()
    dev_logits = torch.empty_like(ring[0])
    h2d = sum(t.numel() * t.element_size() for t in host.values()) + \
        host_logits.numel() * 2 + host_fin.numel()
    d2h = out_tok.numel() * 4 + out_st.numel() * 4 + out_fin.numel()

    def e2e_step():
        idx.trans.copy_(host["trans"], non_blocking=True)
        idx.accept.copy_(host["accept"], non_blocking=True)
        idx.vocab_bytes.copy_(host["vb"], non_blocking=True)
        idx.vocab_offsets.copy_(host["vo"], non_blocking=True)
        dev_logits.copy_(host_logits, non_blocking=True)
        st.copy_(host["states"], non_blocking=True)
        fin.copy_(host_fin, non_blocking=True)
        idx.build()
        idx.step(dev_logits, st, fin, tok)
        out_tok.copy_(tok, non_blocking=True)
        out_st.copy_(st, non_blocking=True)
        out_fin.copy_(fin, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    e2e_steps = max(3, min(args.steps, 50))
    for _ in range(3):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = (time.perf_counter() - t0) / e2e_steps

    def allmax(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    (total_ms, build_ms, mask_ms, mask_in_step_ms, walk_ms_mean, e2e_s, u16_ms, maskonly_ms,
     sample_ms, csr_ms, alias_ms) = map(allmax, (total_ms, build_ms, mask_ms, mask_in_step_ms,
                                                 walk_ms_mean, e2e_s, u16_ms, maskonly_ms, sample_ms,
                                                 csr_ms, alias_ms))
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    walks = float(w.Q) * w.N
    hbm_gbs, peak_kind = load_peaks()
    # ---- bounds derived from this run: SM count, the SM clock sampled under load, and the
    # look-ups per walk the oracle counts on a sample of the states
    threads = len(os.sched_getaffinity(0))
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    sm_hz = 1e6 * float(clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965.0)

    def lookup_bound(wl):
        lpw = lookups_per_walk(wl, threads)
        return sm_count * 32 * sm_hz / lpw, lpw

    def build_modes(wl, t_i32, t_u16, t_mask, rated, why=None):
        n_walks = float(wl.Q) * wl.N
        bound, lpw = lookup_bound(wl)
        out = {
            "Q": wl.Q, "N": wl.N, "walks": n_walks, "sha256": wl.sha256(),
            "lookups_per_walk": lpw,
            "smem_lookup_bound_walks_per_s": bound,
            "bound_inputs": {"sms": sm_count, "lookups_per_clk_per_sm": 32, "sm_mhz": sm_hz / 1e6},
            "int32_states": {"us": t_i32 * 1e3, "walks_per_s": n_walks / (t_i32 * 1e-3),
                             "hbm_write_bound_frac": (n_walks * 4.125 / (t_i32 * 1e-3) / 1e9) / hbm_gbs},
            "uint16_states": {"us": t_u16 * 1e3, "walks_per_s": n_walks / (t_u16 * 1e-3),
                              "hbm_write_bound_frac": (n_walks * 2.125 / (t_u16 * 1e-3) / 1e9) / hbm_gbs},
            "bitmask_only": {"us": t_mask * 1e3, "walks_per_s": n_walks / (t_mask * 1e-3),
                             "smem_lookup_bound_frac": (n_walks / (t_mask * 1e-3)) / bound},
            "rated": rated,
        }
        if why:
            out["note"] = why
        return out

    configs = {}
    if world == 1 and not args.no_configs:
        from fsm_inputs import make_config, step_logits_numpy
        # workload 1: the whole build and 20 greedy steps at B = 1, fp32
        w1 = make_config(1)
        t1 = [time_build(sd, nx, wl=w1) for sd, nx in ((fg.FSM_STATE_I32, True), (fg.FSM_STATE_U16, True),
                                                       (fg.FSM_STATE_I32, False))]
        configs["1_tiny"] = build_modes(w1, *t1, rated=False,
                                        why="6 states x 1,000 tokens: launch latency, not rated")
        i1 = fg.GuidedIndex(w1.dfa.trans, w1.dfa.accept, w1.vocab_bytes, w1.vocab_offsets, w1.dfa.dead,
                            w1.eos_id, device=dev).build()
        x1 = [torch.from_numpy(step_logits_numpy(w1, i)).to(dev) for i in range(w1.steps)]
        s1 = torch.zeros(1, dtype=torch.int32, device=dev)
        f1 = torch.zeros(1, dtype=torch.uint8, device=dev)
        k1 = torch.zeros(1, dtype=torch.int32, device=dev)
        for rep in range(3):
            s1.zero_()
            f1.zero_()
            xs = [x.clone() for x in x1]  # masked in place
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for i in range(w1.steps):
                i1.step(xs[i], s1, f1, k1)
            b.record()
            torch.cuda.synchronize()
        configs["1_tiny"]["greedy_steps"] = {"steps": w1.steps, "B": 1, "dtype": "f32",
                                             "us_per_step": a.elapsed_time(b) / w1.steps * 1e3,
                                             "note": "mask in place, select, advance; launch latency bound"}
        # workload 2: a regular expression's automaton (78 states) over 32,000 tokens
        w2 = make_config(2)
        t2 = [time_build(sd, nx, wl=w2) for sd, nx in ((fg.FSM_STATE_I32, True), (fg.FSM_STATE_U16, True),
                                                       (fg.FSM_STATE_I32, False))]
        configs["2_llama2_json"] = build_modes(
            w2, *t2, rated=False,
            why="2.5 M walks: a microsecond of work behind two launches, launch latency bound, not rated")
        configs["3_llama3_random1k"] = build_modes(w, build_ms, u16_ms, maskonly_ms, rated=True)
        # workload 4: 20,001 states x 152,064 tokens, 12.2 GB of int32 states
        w4 = make_config(4)
        t4 = [time_build(sd, nx, n=3, wl=w4) for sd, nx in ((fg.FSM_STATE_I32, True), (fg.FSM_STATE_U16, True),
                                                            (fg.FSM_STATE_I32, False))]
        configs["4_large_random20k"] = build_modes(
            w4, *t4, rated=True,
            why="the compressed table (2.6 MB) does not fit shared memory: look-ups beyond a row's own "
                "table go through the read-only cache")
        torch.cuda.empty_cache()
    bound3, lpw3 = lookup_bound(w)
    walk_bytes = walks * 4 + w.Q * w.W * 4                    # next-state entries + bitmask words
    live_rows = w.B
    mask_bytes = live_rows * w.N * 2 * 2 + live_rows * w.W * 4
    achieved = walk_bytes / (walk_ms_mean * 1e-3) / 1e9
    mask_achieved = mask_bytes / (mask_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": walks * world / (build_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "index_build_us": build_ms * 1e3, "mask_step_us": mask_ms * 1e3,
        "sample_step_us": sample_ms * 1e3,
        "mask_step_in_step_us": mask_in_step_ms * 1e3, "walk_kernel_us": walk_ms_mean * 1e3,
        "mask_step_loop": {"steps": mask_loop_steps, "live_rows_at_end": rows_live_end,
                           "note": "mask_step_us: back-to-back decode loop over the logits ring; "
                                   "mask_step_in_step_us: the single mask step that follows each "
                                   "index build inside the timed step (shares HBM with the "
                                   "write-back of the index)"},
        "config": config_dict(w, world),
        "roofline": {"bound": "hbm", "kernel": "walk (index build: next-state + bitmask stores)",
                     "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s",
                     "frac": achieved / hbm_gbs, "peak_kind": f"of {peak_kind}",
                     "algorithmic_bytes_per_launch": walk_bytes,
                     "traffic": ncu_traffic("walk_rows")},
        "roofline_mask_step": {"bound": "hbm", "kernel": "mask_step",
                               "achieved": mask_achieved, "peak": hbm_gbs, "unit": "GB/s",
                               "frac": mask_achieved / hbm_gbs, "peak_kind": f"of {peak_kind}",
                               "algorithmic_bytes_per_launch": mask_bytes,
                               "traffic": ncu_traffic("mask_step")},
        "roofline_sample_step": {"bound": "hbm", "kernel": "mask_step (categorical draw)",
                                 "achieved": mask_bytes / (sample_ms * 1e-3) / 1e9, "peak": hbm_gbs,
                                 "unit": "GB/s", "frac": mask_bytes / (sample_ms * 1e-3) / 1e9 / hbm_gbs,
                                 "peak_kind": f"of {peak_kind}",
                                 "algorithmic_bytes_per_launch": mask_bytes, "traffic": None,
                                 "note": "same bytes as the greedy step; the draw adds about 125 "
                                         "integer/fp32 instructions per allowed token"},
        "index_build_modes": {
            "int32_states": {"us": build_ms * 1e3, "walks_per_s": walks / (build_ms * 1e-3),
                             "hbm_write_bound_frac": (walks * 4.125 / (build_ms * 1e-3) / 1e9) / hbm_gbs},
            "uint16_states": {"us": u16_ms * 1e3, "walks_per_s": walks / (u16_ms * 1e-3),
                              "hbm_write_bound_frac": (walks * 2.125 / (u16_ms * 1e-3) / 1e9) / hbm_gbs},
            "bitmask_only": {"us": maskonly_ms * 1e3, "walks_per_s": walks / (maskonly_ms * 1e-3),
                             "smem_lookup_bound_frac": (walks / (maskonly_ms * 1e-3)) / bound3,
                             "note": f"bound = {sm_count} SMs x 32 lookups/clk x {sm_hz / 1e6:.0f} MHz "
                                     f"(sampled under load) / {lpw3:.4f} lookups per walk (oracle-counted "
                                     f"on a sample of states) = {bound3:.3e} walks/s"},
            "compressed_rows": {"us": csr_ms * 1e3, "walks_per_s": walks / (csr_ms * 1e-3),
                                "entries": csr_nnz,
                                "output_bytes": csr_nnz * 8 + (w.Q + 1) * 8 + w.Q * w.W * 4,
                                "note": "fsm_index_build_csr: bitmask + per-state token lists with "
                                        "end states instead of the dense table"},
            "note": "whole builds (all launches), per-rank"},
        "row_merging": {"us": alias_ms * 1e3, "unique_rows": alias_unique,
                        "bytes_read": walk_bytes,
                        "hbm_frac": (walk_bytes / (alias_ms * 1e-3) / 1e9) / hbm_gbs,
                        "note": "fsm_index_row_alias on the int32 index just built: every row hashed "
                                "(one read of bitmask + table), grouped, merges verified exactly"},
        "configs": configs,
        "inputs_sha256": w.sha256(),
        "clocks": clocks,
        "e2e": {"value": walks * world / e2e_s, "unit": UNIT, "ms_per_step": e2e_s * 1e3,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "host DFA, vocabulary, logits and states copied in, tokens/states/finished "
                        "copied out, every step; the index stays on the device for its consumer"},
        "gpu_launches": LAUNCHES_PER_STEP * args.steps,
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, starts)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_sharded(args):
    """`--shard states`: ONE index (workload 4: 20,001 states x 152,064 tokens, int32 states)
    split over the ranks by state slabs.  A step = every rank builds its slab with
    fsm_index_build_rows straight into its place in the full arrays, then the slabs meet in an
    in-place NCCL all-gather (no kernel of this library is handed another rank's memory).
    Strong scaling: the total work is fixed, `value` = Q*N / max-over-ranks step time."""
    import torch
    import paper_2307_09702_b200 as fg
    from paper_2307_09702_b200 import binding, sharding
    from fsm_inputs import make_config

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if fg.fsm_device_check() != 0:
        raise SystemExit("bench.py needs a compute-capability 10.x device")
    fg.fsm_debug_set(binding.FSM_TUNE_WALK_ALGO, args.walk_algo)
    w = make_config(4)
    d = w.dfa
    Q, N, W = d.Q, w.N, (w.N + 31) // 32
    per = -(-Q // world)
    q0, q1 = sharding.equal_slab(Q, rank, world)
    pinned = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a), dtype=dt).pin_memory()
    h_trans, h_acc = pinned(d.trans, torch.int32), pinned(d.accept, torch.uint8)
    h_vb, h_vo = pinned(w.vocab_bytes, torch.uint8), pinned(w.vocab_offsets, torch.int32)
    d_trans, d_acc, d_vb, d_vo = (t.to(dev) for t in (h_trans, h_acc, h_vb, h_vo))
    nbytes = int(w.vocab_offsets[-1])
    full_mask = torch.zeros((world * per, W), dtype=torch.int32, device=dev)
    full_next = torch.zeros((world * per, N), dtype=torch.int32, device=dev)
    wsb = fg.fsm_index_workspace_bytes(Q, N, nbytes)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    h_status = torch.zeros(1, dtype=torch.int32).pin_memory()

    def build():
        if q1 > q0:
            rc = fg.fsm_index_build_rows(d_trans, d_acc, d_vb, d_vo, nbytes, Q, N, d.dead, w.eos_id, q0, q1,
                                         full_mask[q0:q1], full_next[q0:q1], fg.FSM_STATE_I32, ws, wsb, status)
            assert rc == 0, fg.fsm_status_string(rc)

    def gather():
        if dist is not None:
            sharding.all_gather_slabs_in_place(full_mask, Q)
            sharding.all_gather_slabs_in_place(full_next, Q)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        build()
        gather()
    barrier()
    assert int(status.item()) == 0, "data-fault flag raised during warm-up"
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    fg.fsm_debug_set(binding.FSM_PROFILE_WALK, 1)
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    for i in range(args.steps):
        ev[i][0].record()
        build()
        ev[i][1].record()
        gather()
        ev[i][2].record()
    barrier()
    clocks = sampler.stop()
    fg.fsm_debug_set(binding.FSM_PROFILE_WALK, 0)
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    build_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in ev]))
    gather_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in ev]))
    walk = fg.fsm_profile_read()
    walk_ms = float(np.mean(walk)) if walk else build_ms
    # ---- end to end: the inputs come from pinned host memory and the status word goes back
    e2e_steps = max(3, min(args.steps, 50))
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        d_trans.copy_(h_trans, non_blocking=True)
        d_acc.copy_(h_acc, non_blocking=True)
        d_vb.copy_(h_vb, non_blocking=True)
        d_vo.copy_(h_vo, non_blocking=True)
        build()
        gather()
        h_status.copy_(status, non_blocking=True)
        torch.cuda.synchronize()
    barrier()
    e2e_s = (time.perf_counter() - t0) / e2e_steps

    def allmax(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    total_ms, build_ms, gather_ms, walk_ms, e2e_s = map(allmax, (total_ms, build_ms, gather_ms, walk_ms, e2e_s))
    # ---- every rank checks sampled rows of the gathered index (its own slab and the others')
    # against the CPU oracle
    from oracle import fsm_oracle
    for q in sorted({0, q0, max(q0, q1 - 1), (q0 + 7919) % Q, Q - 1, (Q // 2 + 1000 * rank) % Q}):
        m, n, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                                         q_begin=q, q_end=q + 1, threads=len(os.sched_getaffinity(0)))
        assert (full_mask[q].cpu().numpy().view(np.uint32) == m[0]).all(), q
        assert (full_next[q].cpu().numpy() == n[0]).all(), q
    if rank != 0:
        dist.destroy_process_group()
        return
    hbm_gbs, peak_kind = load_peaks()
    walks = float(Q) * N
    step_ms = total_ms / args.steps
    slab_bytes = (q1 - q0) * (N * 4 + W * 4)
    achieved = slab_bytes / (walk_ms * 1e-3) / 1e9
    moved = (world - 1) * per * (N + W) * 4          # bytes every rank receives per step
    h2d = sum(t.numel() * t.element_size() for t in (h_trans, h_acc, h_vb, h_vo))
    line = {
        "metric": METRIC, "value": walks / (step_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "slab_build_us": build_ms * 1e3, "walk_kernel_us": walk_ms * 1e3, "allgather_us": gather_ms * 1e3,
        "allgather_gbs_per_rank": (moved / (gather_ms * 1e-3) / 1e9) if world > 1 and gather_ms > 0 else None,
        "config": {"workload": "4_large_random20k: ONE index, random DFA Q=20001 x Qwen2-shaped vocab "
                               "N=152064, int32 next-state + packed bitmask, split over the ranks by "
                               "state slabs and all-gathered (NCCL, in place)",
                   "Q": Q, "N": N, "state_dtype": "int32", "shard": "states",
                   "rows_per_rank": per, "parallelism": f"state slabs x{world} + all-gather",
                   "l2": "outputs larger than L2: every rank writes its slab of the 12.2 GB index"},
        "roofline": {"bound": "hbm", "kernel": "walk (index build: next-state + bitmask stores)",
                     "achieved": achieved, "peak": hbm_gbs, "unit": "GB/s", "frac": achieved / hbm_gbs,
                     "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": slab_bytes,
                     "traffic": None},
        "inputs_sha256": w.sha256(),
        "checked": "sampled rows of the gathered index equal the CPU oracle on every rank",
        "clocks": clocks,
        "e2e": {"value": walks / e2e_s, "unit": UNIT, "ms_per_step": e2e_s * 1e3,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 4,
                "note": "automaton and vocabulary copied in from pinned host memory, status word "
                        "copied out, every step; the index stays on the devices"},
        "gpu_launches": 2 * args.steps,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_only_build(args):
    """A small case for profilers: builds workload K (optionally only the state slab
    q0..q1-1, through fsm_index_build_rows) a few times and prints its time."""
    import torch
    import paper_2307_09702_b200 as fg
    from paper_2307_09702_b200 import binding
    from fsm_inputs import make_config
    parts = args.only_build.split(":")
    k = int(parts[0])
    w = make_config(k)
    d = w.dfa
    q0, q1 = (int(parts[1]), int(parts[2])) if len(parts) == 3 else (0, d.Q)
    torch.cuda.set_device(0)
    fg.fsm_debug_set(binding.FSM_TUNE_WALK_ALGO, args.walk_algo)
    modes = {"int32": (fg.FSM_STATE_I32, True), "uint16": (fg.FSM_STATE_U16, True),
             "bitmask": (fg.FSM_STATE_I32, False)}
    sd, want_next = modes[args.build_mode]
    idx = fg.GuidedIndex(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id, sd,
                         want_next, q_begin=q0, q_end=q1)
    for _ in range(args.warmup):
        idx.build()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for _ in range(args.steps):
        idx.build()
    b.record()
    torch.cuda.synchronize()
    assert int(idx.status.item()) == 0
    us = a.elapsed_time(b) / args.steps * 1e3
    print(json.dumps({"only_build": args.only_build, "mode": args.build_mode, "rows": q1 - q0, "N": w.N,
                      "us": us, "walks_per_s": (q1 - q0) * w.N / (us * 1e-6)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the per-workload block (workloads 1, 2 and 4)")
    ap.add_argument("--walk-algo", type=int, default=0, choices=[0, 1, 2, 3],
                    help="index walk: 0 automatic, 1 dense warp-tile, 2 row-wise work-avoiding, "
                         "3 bucket walk (bitmask-only builds)")
    ap.add_argument("--only-build", default=None, metavar="K[:Q0:Q1]",
                    help="profiling aid: only build workload K (or its state slab Q0..Q1-1) "
                         "--steps times after --warmup builds")
    ap.add_argument("--build-mode", default="int32", choices=["int32", "uint16", "bitmask"])
    ap.add_argument("--shard", default="none", choices=["none", "states"],
                    help="states: split ONE workload-4 index over the ranks by state slabs and "
                         "all-gather it (strong scaling) instead of one independent problem per rank")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.only_build:
        run_only_build(args)
        return
    if args.impl == "reference":
        run_reference(args)
    elif args.shard == "states":
        args.steps = min(args.steps, 300)      # a step writes 12.2 GB
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
