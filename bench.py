#!/usr/bin/env python
"""Benchmark of the constrained decoding step (and the token-table build).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  A "step" is one constrained decoding step (mask from
state, -inf penalty, arg-max, next state) for the whole batch of the
``string_256k`` workload: vocabulary 256,000 x batch 512, fp32 logits,
8,195-state string-literal DFA.  Logits cycle through a pool of seeded
tensors, each larger than the L2 cache; rows that finish are restarted at the
start state so every row stays active.  With N > 1 every rank runs an
independent replica (the path has no exchange step).

``--impl reference`` times the CPU oracle on the same workload instead.
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

import numpy as np  # noqa: E402

WORKLOAD = "string_256k"
METRIC = "constrained_step_logits_per_s"
UNIT = "logits/s"
POOL = 4
BYTES_PER_LOGIT_F32_GREEDY = 4 + 4 + 1.0 / 8.0    # read + masked write + mask bit
BYTES_PER_TRANSITION = 2 + 1.0 / 8.0              # int16 next entry + mask bit, stores only
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum and dram__bytes_write.sum of one step launch of the small profiling case
# (`--case small`: 128 rows x 256,000 fp32 logits), from the ncu capture summarised in
# profiles/step_vec_kernel_fp32_small_case.md, with the SHA-256 of the kernel source the
# capture ran.  Reads grow in proportion to the logits per launch; writes are the algorithmic
# bytes less what is still in L2 when the kernel ends (the same ~53 MB at any size).  The bench
# reports null when the source has changed since the capture.
STEP_TRAFFIC_SMALL_CASE_READ_BYTES = 133925376.0
STEP_TRAFFIC_SMALL_CASE_WRITE_BYTES = 78181632.0
STEP_TRAFFIC_SMALL_CASE_LOGITS = 128 * 256000
STEP_TRAFFIC_SOURCE_SHA256 = "b97172796b39aa93f7182c74308a3184f0e9afbb37beeff71bcb395fdce9b03e"
STEP_KERNEL_SOURCE = os.path.join(ROOT, "paper_2407_08103_b200", "csrc", "cstr_step.cu")


def file_sha256(path: str) -> str:
    import hashlib
    with open(path, "rb") as fh:
        return hashlib.sha256(fh.read()).hexdigest()


def step_traffic_bytes(logits_per_launch: int):
    """DRAM traffic of one fp32 greedy step launch, from the recorded small-case capture; None
    when there is no capture or the step kernel's source is no longer the captured one."""
    if STEP_TRAFFIC_SMALL_CASE_READ_BYTES is None or STEP_TRAFFIC_SOURCE_SHA256 is None:
        return None
    try:
        if file_sha256(STEP_KERNEL_SOURCE) != STEP_TRAFFIC_SOURCE_SHA256:
            return None
    except OSError:
        return None
    scale = logits_per_launch / STEP_TRAFFIC_SMALL_CASE_LOGITS
    in_l2_at_end = STEP_TRAFFIC_SMALL_CASE_LOGITS * 4 - STEP_TRAFFIC_SMALL_CASE_WRITE_BYTES
    return STEP_TRAFFIC_SMALL_CASE_READ_BYTES * scale + max(logits_per_launch * 4 - in_l2_at_end, 0.0)


def roofline_entry(achieved_gbs: float, peak: float, peak_kind: str, bound: str = "hbm",
                   traffic=None, **extra):
    """A roofline object: achieved algorithmic GB/s against the measured copy rate and,
    beside it, against the nominal 8 TB/s."""
    d = {"bound": bound, "achieved": achieved_gbs, "peak": peak, "unit": "GB/s",
         "frac": achieved_gbs / peak, "traffic": traffic, "peak_kind": "of %s" % peak_kind,
         "frac_of_nominal_8TBs": achieved_gbs / NOMINAL_HBM_GBS}
    d.update(extra)
    return d


def time_copy_of(torch, n_bytes_moved: int, dev, stream, reps: int = 12) -> float:
    """Milliseconds a plain device copy (torch ``copy_``, one read and one write stream) takes
    to move `n_bytes_moved` bytes in total: what launch, ramp-up and tail cost ANY kernel of
    that size on this GPU, the measured copy peak being quoted on a 4 GB copy.  Source and
    destination alternate between two pairs, each pair larger than the L2 where possible."""
    n = max(int(n_bytes_moved) // 8, 1)                # fp32 elements: 4 bytes read + 4 written
    pairs = [(torch.empty(n, dtype=torch.float32, device=dev).normal_(),
              torch.empty(n, dtype=torch.float32, device=dev)) for _ in range(2)]
    ms = []
    for i in range(reps + 3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        src, dst = pairs[i & 1]
        a.record(stream)
        dst.copy_(src)
        b.record(stream)
        b.synchronize()
        if i >= 3:
            ms.append(a.elapsed_time(b))
    return float(np.mean(ms))


def inputs_sha256(dfa, vb, vo, first_logits_row) -> str:
    """One digest over the seeded inputs (DFA table, accept flags, vocabulary, first logits
    row), so that two bench lines can be seen to have run on the same data."""
    import hashlib
    h = hashlib.sha256()
    for a in (dfa[0], dfa[1], vb, vo, first_logits_row):
        h.update(np.ascontiguousarray(a).tobytes())
    return h.hexdigest()


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2560)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=12.0,
                    help="CPU time budget of the oracle baseline leg")
    ap.add_argument("--case", default="full", choices=["full", "small"],
                    help="small: batch 128 and a 4,099-state string-literal DFA over the same "
                         "vocabulary (for profiler captures); its numbers are not bench values")
    ap.add_argument("--skip-build-bench", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-other-workloads", action="store_true",
                    help="do not time the four other workloads (reported under 'other_workloads')")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--build-only", default=None, metavar="WORKLOAD",
                    help="time only the token-table build of one workload (with --case small: the "
                         "4,099-state string DFA / a 4,096-state random DFA; small_constraints: the five "
                         "small-constraint compiles over the 256,000-token vocabulary; wildcard: the "
                         "terminal-label build; random9728_128k: a 9,728-state random DFA over the "
                         "128,256-token vocabulary, which takes the staged-rows builder) and print its entry; "
                         "for profiler captures, not a bench line")
    ap.add_argument("--walker", default="trie", choices=["trie", "dense"],
                    help="with --build-only: trie = cstr_table_build, dense = cstr_table_build_dense "
                         "(every token from its first byte; the baseline the trie walk is compared with)")
    ap.add_argument("--step-only", default=None, metavar="VARIANT",
                    choices=["f32", "bf16", "f32_noise", "bf16_noise", "scalar", "speculative"],
                    help="time only one instantiation of the step on the small profiling case (128 rows "
                         "x 256,000 tokens, 4,099-state string DFA): the vector kernel for fp32 / bf16 "
                         "logits without / with a noise stream, the scalar kernel (row stride not a "
                         "multiple of 16 bytes), or the speculative-verification pair; for profiler "
                         "captures, not a bench line")
    ap.add_argument("--download-only", action="store_true",
                    help="time only cstr_table_download of a 256-state slab of the small string table "
                         "(device-side decode + transpose, one copy to the host); for profiler captures")
    ap.add_argument("--pushdown-only", action="store_true",
                    help="time only the push-down step leg (batch 128 with --case small) and print "
                         "its entry; for profiler captures, not a bench line")
    return ap.parse_args()


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def workload_inputs(case: str = "full"):
    """Seeded host inputs of the benchmark workload: recipe, DFA, vocabulary."""
    import dataclasses
    from synth.configs import CONFIGS, config_dfas, config_vocab
    w = CONFIGS[WORKLOAD]
    vb, vo = config_vocab(WORKLOAD)
    if case == "small":
        from synth.regex_frontend import regex_to_dfa
        w = dataclasses.replace(w, batch=128)
        dfa = regex_to_dfa(w.regex.replace("{0,4096}", "{0,2048}"))
    else:
        dfa = config_dfas(WORKLOAD)[0]
    return w, dfa, vb, vo


def global_rows(rank: int, batch: int):
    """Row ids of this replica: every rank decodes its own `batch` rows (weak scaling)."""
    return range(rank * batch, rank * batch + batch)


def reduce_max(x: float, world: int, device) -> float:
    """Maximum of a per-rank number over all ranks (the slowest rank sets the time)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_step: int, world: int, steps: int, max_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's device time."""
    return units_per_rank_step * world * steps / (max_ms * 1e-3)


class ClockSampler(threading.Thread):
    """Polls SM clock, power and clock-event reasons through NVML (read-only)."""

    def __init__(self, device_index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples = []      # (t, sm_mhz, reasons_bitmask, power_w)
        self.stop_flag = threading.Event()
        self.ok = False
        self.sm_max = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:  # pragma: no cover - depends on the box
            self.err = repr(exc)

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                sm = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                pw = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.samples.append((time.perf_counter(), sm, rs, pw))
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self, t0: float, t1: float):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["unavailable"]}
        nv = self.nv
        sel = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(sel) < 3:
            sel, window = self.samples, "whole run (timed region shorter than 3 samples)"
        names = {
            nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksEventReasonHwPowerBrakeSlowdown: "hw_power_brake_slowdown",
            nv.nvmlClocksEventReasonApplicationsClocksSetting: "applications_clocks_setting",
            nv.nvmlClocksEventReasonSyncBoost: "sync_boost",
        }
        seen = 0
        for s in sel:
            seen |= s[2]
        reasons = [n for bit, n in names.items() if seen & bit]
        return {"sm_mhz": float(np.median([s[1] for s in sel])), "sm_max_mhz": self.sm_max,
                "reasons": reasons, "power_w_max": max(s[3] for s in sel), "samples": len(sel),
                "window": window}


def cpu_model_string() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def time_oracle_single_thread(dfa, vb, vo, pool, rows: int = 8):
    """The oracle on one thread: `rows` rows of one step (logits/s)."""
    import oracle
    states = np.full(rows, dfa[2], dtype=np.int32)
    t0 = time.perf_counter()
    oracle.step([dfa], vb, vo, pool[:rows], states, threads=1)
    return rows * pool.shape[1] / (time.perf_counter() - t0)


def time_oracle_table_build(dfa, vb, vo, budget_s: float = 3.0):
    """The oracle's token table for slabs of states (all host threads) until the
    budget is used: transitions/s, with what was timed."""
    import oracle
    threads = oracle.max_threads()
    S, V = int(dfa[0].shape[0]), vo.size - 1
    slab = min(S, 4 * threads)
    oracle.token_table(dfa[0], dfa[1], vb, vo, q_lo=0, q_hi=min(S, threads), threads=threads)  # warm
    done, t0 = 0, time.perf_counter()
    while done < S and (done == 0 or time.perf_counter() - t0 < budget_s):
        hi = min(S, done + slab)
        oracle.token_table(dfa[0], dfa[1], vb, vo, q_lo=done, q_hi=hi, threads=threads)
        done = hi
    dt = time.perf_counter() - t0
    return {"value": done * V / dt, "unit": "transitions/s", "cores": threads, "kind": "oracle",
            "sample": "%d of %d states x %d tokens of %s in %.1f s (whole table extrapolates to "
                      "%.1f s)" % (done, S, V, WORKLOAD, dt, S * V / (done * V / dt))}


def time_oracle(w, dfa, vb, vo, pools, budget_s: float, max_steps: int):
    """The oracle as it stands, all host threads, whole-batch steps until the
    time budget is used (at least 2 steps).  Returns (logits/s, cores, sample text, s/step)."""
    import oracle
    threads = oracle.max_threads()
    B, V = pools[0].shape
    states = np.full(B, dfa[2], dtype=np.int32)
    oracle.step([dfa], vb, vo, pools[0][:8], states[:8], threads=threads)   # load + warm
    done, t0 = 0, time.perf_counter()
    while done < max_steps and (done < 2 or time.perf_counter() - t0 < budget_s):
        res = oracle.step([dfa], vb, vo, pools[done % len(pools)], states, threads=threads)
        states = np.where(res["states"] < 0, dfa[2], res["states"]).astype(np.int32)
        done += 1
    dt = time.perf_counter() - t0
    sample = "%d whole-batch steps (%d rows x %d tokens) of %s, %.1f s" % (done, B, V, WORKLOAD, dt)
    return B * V * done / dt, threads, sample, dt / done


def time_other_workload(name, torch, cstr, ConstrainedDecoder, dev, stream, peak, peak_kind,
                        steps=48):
    """Step-kernel and table-build timing of one of the other workloads: device
    generated seeded logits (timing only; parity is covered by the tests), a
    pool of tensors larger than twice the L2 where the batch allows, finished
    rows restarted, events around each step launch."""
    from synth.configs import CONFIGS, config_dfas, config_vocab, row_table_for
    w = CONFIGS[name]
    dfas = config_dfas(name)
    vb, vo = config_vocab(name)
    V, B = vo.size - 1, w.batch
    vocab = cstr.cstr_load_vocab(vb, vo)
    tables, handles, build_ms = [], [], []
    for d in dfas:
        h = cstr.cstr_load_dfa(*d)
        t = cstr.cstr_table_create(vocab, d[0].shape[0])
        for rep in range(3 if len(tables) == 0 else 1):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            cstr.cstr_table_build(t, h, -1, stream)
            a1.record(stream)
            a1.synchronize()
            if len(tables) == 0 and rep > 0:
                build_ms.append(a0.elapsed_time(a1))
        tables.append(t)
        handles.append(h)
    esz = 4 if w.dtype == "f32" else 2
    tdtype = torch.float32 if w.dtype == "f32" else torch.bfloat16
    tensor_bytes = B * V * esz
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    pool_n = int(max(2, min(256, -(-2 * l2 // tensor_bytes))))
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.logits_seed)
    pool = [(torch.randn((B, V), generator=gen, device=dev, dtype=torch.float32) * w.sigma).to(tdtype)
            for _ in range(pool_n)]
    noise = None
    if w.gumbel:
        gen.manual_seed(w.noise_seed)
        noise = []
        for _ in range(min(pool_n, 2)):
            u = torch.rand((B, V), generator=gen, device=dev, dtype=torch.float32).clamp_(1e-20, 1 - 1e-7)
            noise.append(-torch.log(-torch.log(u)))
    row_table = row_table_for(w, B)
    dec = ConstrainedDecoder(tables, B, row_table=row_table, device=dev)
    start_vec = dec.states.clone()
    out = [torch.empty((B, V), dtype=tdtype, device=dev) for _ in range(2)]
    pairs = []
    for i in range(steps + 4):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        dec.step(pool[i % pool_n], noise=None if noise is None else noise[i % len(noise)],
                 masked_out=out[i & 1], stream=stream)
        e1.record(stream)
        torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)
        if i >= 4:
            pairs.append((e0, e1))
    torch.cuda.synchronize()
    kernel_ms = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
    # the same steps back to back between one pair of events (restart op included):
    # for the small workloads this, not the per-launch bracket, is the sustained cost
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    loop_steps = 200
    l0.record(stream)
    for i in range(loop_steps):
        dec.step(pool[i % pool_n], noise=None if noise is None else noise[i % len(noise)],
                 masked_out=out[i & 1], stream=stream)
        torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)
    l1.record(stream)
    l1.synchronize()
    loop_ms = l0.elapsed_time(l1) / loop_steps
    # and as one CUDA graph of 32 steps (cstr_step only enqueues kernels, so a
    # sampling loop can be captured): removes the host launch cost that
    # dominates the small workloads
    def graph_time(rotate):
        """32 steps per graph; rotate=False keeps one logits tensor (L2-resident when it fits)."""
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            dec.step(pool[0], noise=None if noise is None else noise[0], masked_out=out[0])
            with torch.cuda.graph(g, stream=side):
                for i in range(32):
                    k = i % pool_n if rotate else 0
                    dec.step(pool[k], noise=None if noise is None else noise[k % len(noise)],
                             masked_out=out[i & 1])
                    torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)
            g.replay()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(side)
            for _ in range(8):
                g.replay()
            g1.record(side)
            g1.synchronize()
        stream.wait_stream(side)
        return g0.elapsed_time(g1) / (8 * 32)

    graph_ms = graph_resident_ms = None
    try:
        graph_ms = graph_time(True)
        graph_resident_ms = graph_time(False)
    except Exception as exc:  # pragma: no cover - depends on the box
        sys.stderr.write("graph timing of %s skipped: %r\n" % (name, exc))
    # the same table by the per-token walker without the trie (the pair "trie vs dense")
    dense = []
    for _ in range(3):
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        cstr.cstr_table_build_dense(tables[0], handles[0], -1, stream)
        a1.record(stream)
        a1.synchronize()
        dense.append(a0.elapsed_time(a1))
    dense_ms = float(np.mean(dense[1:]))
    bytes_per_logit = 2 * esz + (4 if w.gumbel else 0) + 1.0 / 8.0
    step_bytes = B * V * bytes_per_logit
    gbs = step_bytes / (kernel_ms * 1e-3) / 1e9
    S0 = int(dfas[0][0].shape[0])
    bms = float(np.mean(build_ms))
    bgbs = S0 * V * BYTES_PER_TRANSITION / (bms * 1e-3) / 1e9
    hbm_honest = pool_n * tensor_bytes >= 2 * l2
    copy_ms = time_copy_of(torch, step_bytes, dev, stream) if hbm_honest else None
    return {
        "workload": name, "vocab": V, "batch": B, "dfa_states": [int(d[0].shape[0]) for d in dfas],
        "dtype": w.dtype, "sampler": "gumbel-max" if w.gumbel else "greedy",
        "tables": len(tables), "step_kernel_ms": kernel_ms, "step_loop_ms": loop_ms,
        "step_graph_ms": graph_ms, "step_graph_ms_same_tensor": graph_resident_ms,
        "logits_per_s": B * V / (kernel_ms * 1e-3),
        "roofline": roofline_entry(
            gbs, peak, peak_kind,
            bound="hbm" if hbm_honest else "launch latency (working set sits in L2)",
            bytes_per_logit=bytes_per_logit,
            logits_pool="%d tensors x %.1f MB" % (pool_n, tensor_bytes / 1e6),
            same_size_copy_ms=copy_ms,
            frac_of_same_size_copy=None if copy_ms is None else copy_ms / kernel_ms),
        "table_build": {"dfa_states": S0, "ms": bms, "transitions_per_s": S0 * V / (bms * 1e-3),
                        "dense_walker_ms": dense_ms,
                        "roofline": roofline_entry(bgbs, peak, peak_kind,
                                                   note="stores of next + mask only")},
    }


def time_wildcard_build(torch, cstr, vocab, vb, vo, stream, peak, peak_kind):
    """Table build of a constraint with terminal-label (wildcard) edges over the
    256k vocabulary: the paper's bulleted-summary example (Section 2.5.1), with
    PARAGRAPH_TOKEN = the newline-free tokens."""
    from synth.regex_frontend import regex_to_dfa
    full = regex_to_dfa(r"Summary:(\n\* (?P<PARAGRAPH_TOKEN>)+){3,5}", ["PARAGRAPH_TOKEN"])
    trans, term = np.ascontiguousarray(full[0][:, :256]), np.ascontiguousarray(full[0][:, 256:])
    V = vo.size - 1
    has_nl = np.zeros(V, dtype=bool)
    has_nl[np.searchsorted(vo, np.nonzero(vb == 0x0A)[0], side="right") - 1] = True
    cstr.cstr_vocab_set_token_sets(vocab, (~has_nl).astype(np.uint32), 1)
    h = cstr.cstr_load_dfa_terminals(trans, term, full[1], full[2])
    S = int(trans.shape[0])
    t = cstr.cstr_table_create(vocab, S)
    ms = []
    for _ in range(4):
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        cstr.cstr_table_build(t, h, -1, stream)
        a1.record(stream)
        a1.synchronize()
        ms.append(a0.elapsed_time(a1))
    best = float(np.mean(ms[1:]))
    return {"workload": "summary bullets with PARAGRAPH_TOKEN wildcard x vocab 256,000",
            "dfa_states": S, "states_with_terminal_edges": int((term >= 0).any(axis=1).sum()),
            "ms": best, "transitions_per_s": S * V / (best * 1e-3),
            "roofline": roofline_entry(S * V * BYTES_PER_TRANSITION / (best * 1e-3) / 1e9, peak,
                                       peak_kind, bound="launch latency (tens of microseconds)",
                                       note="stores of next + mask only")}


def time_pushdown(torch, cstr, PushdownDecoder, dev, stream, peak, peak_kind, V=256000, B=512,
                  steps=48):
    """Push-down step (Algorithm 3) on a nested-JSON PDA over a 256,000-token
    vocabulary with structural multi-bracket tokens, batch 512, fp32, greedy:
    table build (allocation + kernel) and the two-kernel step (situation
    lookup; fused penalise / select / edge traversal), events around each call;
    finished rows are restarted."""
    from synth import json_pda, make_vocab_json
    P = json_pda(space=True)
    vb, vo = make_vocab_json(V, seed=0)
    vocab = cstr.cstr_load_vocab(vb, vo)
    h = cstr.cstr_load_pda(P.src, P.inp, P.tgt, P.pop_off, P.pops, P.push_off, P.pushes, P.accept,
                           P.n_symbols, P.start)
    t0 = time.perf_counter()
    table = cstr.cstr_build_pda_table(h, vocab, -1, stream)        # allocation + first build
    torch.cuda.synchronize()
    create_ms = (time.perf_counter() - t0) * 1e3
    build_ms = []
    for _ in range(4):                                              # the build kernels alone
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        cstr.cstr_pda_table_rebuild(table, -1, stream)
        a1.record(stream)
        a1.synchronize()
        build_ms.append(a0.elapsed_time(a1))
    build_ms = build_ms[1:]
    n_cfg = P.n_states * (P.n_symbols + 1)
    gen = torch.Generator(device=dev)
    gen.manual_seed(17)
    pool = [torch.randn((B, V), generator=gen, device=dev) for _ in range(3)]
    out = [torch.empty((B, V), device=dev) for _ in range(2)]
    dec = PushdownDecoder(table, B, stack_cap=64, device=dev)
    pairs = []
    for i in range(steps + 4):                      # no host synchronisation inside the loop
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        dec.step(pool[i % 3], masked_out=out[i & 1], stream=stream)
        e1.record(stream)
        dec.restart_finished()
        if i >= 4:
            pairs.append((e0, e1))
    torch.cuda.synchronize()
    ms = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
    depth_sum, depth_max, probes = 0.0, 0, 8        # stack statistics, outside the timing
    for i in range(probes):
        dec.step(pool[i % 3], masked_out=out[i & 1], stream=stream)
        dec.restart_finished()
        depth_sum += float(dec.depths.float().mean().item())
        depth_max = max(depth_max, int(dec.depths.max().item()))
    bad, empty, overflow = dec.status()
    gbs = B * V * BYTES_PER_LOGIT_F32_GREEDY / (ms * 1e-3) / 1e9
    return {"workload": "nested JSON PDA (%d states, %d stack symbols, %d situations) x vocab %d, "
                        "batch %d, fp32 greedy" % (P.n_states, P.n_symbols, n_cfg, V, B),
            "table_build_ms": float(np.mean(build_ms)), "table_create_and_build_ms": create_ms,
            "table_transitions_per_s": n_cfg * V / (float(np.mean(build_ms)) * 1e-3),
            "step_ms": ms, "logits_per_s": B * V / (ms * 1e-3),
            "roofline": roofline_entry(gbs, peak, peak_kind,
                                       note="two kernels per step (situation lookup, fused step); "
                                            "8.125 algorithmic bytes per logit"),
            "mean_stack_depth": depth_sum / probes, "max_stack_depth": depth_max,
            "status_rows": {"bad": bad, "empty_mask": empty, "overflow": overflow}}


def time_build_only(torch, cstr, name, case, stream, repeats=4, walker="trie"):
    """Token-table build of one workload's (first) DFA over its vocabulary."""
    from synth import random_range_dfa
    from synth.configs import CONFIGS, config_dfas, config_vocab
    from synth.regex_frontend import regex_to_dfa
    w = CONFIGS.get(name)
    vb, vo = config_vocab(name) if name in CONFIGS else (None, None)
    if case == "small" and name == "string_256k":
        dfa = regex_to_dfa(w.regex.replace("{0,4096}", "{0,2048}"))
    elif case == "small" and name == "random10k_256k":
        dfa = random_range_dfa(4096, seed=2)
    elif name == "random9728_128k":          # the staged-rows builder at a profiler-friendly size
        w = CONFIGS["random10k_256k"]
        vb, vo = config_vocab("schema40_128k")
        dfa = random_range_dfa(9728, seed=2)
    else:
        dfa = config_dfas(name)[0]
    V, S = vo.size - 1, int(dfa[0].shape[0])
    vocab = cstr.cstr_load_vocab(vb, vo)
    h = cstr.cstr_load_dfa(*dfa)
    table = cstr.cstr_table_create(vocab, S)
    ms = []
    for _ in range(repeats):
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        if walker == "dense":
            cstr.cstr_table_build_dense(table, h, -1, stream)
        else:
            cstr.cstr_table_build(table, h, -1, stream)
        a1.record(stream)
        a1.synchronize()
        ms.append(a0.elapsed_time(a1))
    best = float(np.mean(ms[1:]))
    peak, kind = measured_hbm_peak()
    gbs = S * V * BYTES_PER_TRANSITION / (best * 1e-3) / 1e9
    return {"workload": name + (" (small case)" if case == "small" else ""), "walker": walker,
            "dfa_states": S, "vocab": V, "ms": best, "transitions_per_s": S * V / (best * 1e-3),
            "roofline": roofline_entry(gbs, peak, kind, note="stores of next + mask only")}


def time_step_variant(torch, cstr, variant, dev, stream, steps=12):
    """One instantiation of the step kernel on the small profiling case."""
    from synth.configs import config_vocab
    from synth.regex_frontend import regex_to_dfa
    from synth.constraints import STRING_LITERAL_REGEX
    vb, vo = config_vocab(WORKLOAD)
    V, B = vo.size - 1, 128
    dfa = regex_to_dfa(STRING_LITERAL_REGEX.replace("{0,4096}", "{0,2048}"))
    vocab = cstr.cstr_load_vocab(vb, vo)
    table = cstr.cstr_table_create(vocab, dfa[0].shape[0])
    cstr.cstr_table_build(table, cstr.cstr_load_dfa(*dfa), -1, stream)
    bf16 = variant.startswith("bf16")
    noise_on = variant.endswith("noise")
    ld = V + 1 if variant == "scalar" else V          # an odd stride takes the scalar kernel
    tdtype = torch.bfloat16 if bf16 else torch.float32
    gen = torch.Generator(device=dev)
    gen.manual_seed(11)
    pool = [torch.randn((B, ld), generator=gen, device=dev).to(tdtype) for _ in range(3)]
    noise = None
    if noise_on:
        u = torch.rand((B, ld), generator=gen, device=dev).clamp_(1e-20, 1 - 1e-7)
        noise = -torch.log(-torch.log(u))
    out = torch.empty((B, ld), dtype=tdtype, device=dev)
    ws = cstr.cstr_workspace_create(B)
    start = torch.full((B,), int(dfa[2]), dtype=torch.int32, device=dev)
    st = start.clone()
    st_out = torch.empty_like(st)
    tok = torch.empty(B, dtype=torch.int32, device=dev)
    kk, seqs = 7, B // 8
    draft = torch.zeros((seqs, kk), dtype=torch.int32, device=dev)
    n_acc = torch.empty(seqs, dtype=torch.int32, device=dev)
    out_tok = torch.empty((seqs, kk + 1), dtype=torch.int32, device=dev)
    new_st = torch.empty(seqs, dtype=torch.int32, device=dev)
    ms = []
    for i in range(steps + 3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        if variant == "speculative":
            cstr.cstr_step_history([table], pool[i % 3][:, :V], st, st_out, tok, out[:, :V], ws,
                                   stream=stream)
            cstr.cstr_accept_draft(draft, tok.view(seqs, kk + 1), st_out.view(seqs, kk + 1), n_acc,
                                   out_tok, new_st, stream=stream)
        else:
            cstr.cstr_step([table], pool[i % 3][:, :V], st, tok, out[:, :V], ws, noise=None if noise
                           is None else noise[:, :V], stream=stream)
            torch.where(st < 0, start, st, out=st)
        b.record(stream)
        b.synchronize()
        if i >= 3:
            ms.append(a.elapsed_time(b))
    best = float(np.mean(ms))
    esz = 2 if bf16 else 4
    bpl = 2 * esz + (4 if noise_on else 0) + 1.0 / 8.0
    peak, kind = measured_hbm_peak()
    return {"variant": variant, "batch": B, "vocab": V, "row_stride": ld, "ms": best,
            "roofline": roofline_entry(B * V * bpl / (best * 1e-3) / 1e9, peak, kind,
                                       bytes_per_logit=bpl)}


def time_small_compiles(torch, cstr, vocab, stream):
    """Compile cost of small constraints over the 256k vocabulary (the regime of the
    paper's Table 1: one small regex against a large vocabulary): table build
    kernels alone, and DFA load + build end to end on the host clock."""
    from synth import constraints
    from synth.regex_frontend import regex_to_dfa
    pats = dict(constraints.SMALL_CONSTRAINTS)
    pats["api_call"] = constraints.API_CALL_REGEX
    pats["flat_json"] = constraints.FLAT_JSON_REGEX
    out = []
    for name, pat in pats.items():
        dfa = regex_to_dfa(pat)
        S = int(dfa[0].shape[0])
        h = cstr.cstr_load_dfa(*dfa)
        t = cstr.cstr_table_create(vocab, S)
        ms = []
        for _ in range(4):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            cstr.cstr_table_build(t, h, -1, stream)
            a1.record(stream)
            a1.synchronize()
            ms.append(a0.elapsed_time(a1))
        e2e = []
        for _ in range(3):
            t0 = time.perf_counter()
            h2 = cstr.cstr_load_dfa(*dfa)
            cstr.cstr_table_build(t, h2, -1, stream)
            torch.cuda.synchronize()
            e2e.append((time.perf_counter() - t0) * 1e3)
        out.append({"constraint": name, "dfa_states": S, "build_ms": float(np.mean(ms[1:])),
                    "dfa_load_plus_build_ms": float(min(e2e))})
    return out


def time_small_batches(torch, cstr, table, V, dev, stream, batches=(1, 8, 64)):
    """Step latency for small batches at the full vocabulary (fp32, greedy): 64
    steps captured in one CUDA graph, logits rotating through a pool larger than
    the L2 where it fits in 300 MB, states held constant (state-history form)."""
    out = []
    gen = torch.Generator(device=dev)
    gen.manual_seed(5)
    for B in batches:
        n_pool = max(2, min(64, 300_000_000 // (B * V * 4)))
        pool = [torch.randn((B, V), generator=gen, device=dev) for _ in range(n_pool)]
        masked = torch.empty((B, V), device=dev)
        st_in = torch.full((B,), 5, dtype=torch.int32, device=dev)
        st_out, tok = torch.empty_like(st_in), torch.empty_like(st_in)
        ws = cstr.cstr_workspace_create(B)
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(stream)
        try:
            with torch.cuda.stream(side):
                cstr.cstr_step_history([table], pool[0], st_in, st_out, tok, masked, ws)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    for i in range(64):
                        cstr.cstr_step_history([table], pool[i % n_pool], st_in, st_out, tok, masked, ws)
                g.replay()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(side)
                for _ in range(10):
                    g.replay()
                e1.record(side)
                e1.synchronize()
            us = e0.elapsed_time(e1) / 640 * 1e3
            out.append({"batch": B, "us_per_step": us,
                        "gb_per_s": B * V * BYTES_PER_LOGIT_F32_GREEDY / us / 1e3,
                        "logits_pool": n_pool})
        except Exception as exc:  # pragma: no cover - depends on the box
            sys.stderr.write("small-batch timing skipped: %r\n" % (exc,))
        stream.wait_stream(side)
        del pool
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from synth import normal_logits
    w, dfa, vb, vo = workload_inputs(args.case)
    V = vo.size - 1
    B = w.batch
    import oracle
    oracle.build()
    pools = [normal_logits(w.logits_seed, k, range(B), V) for k in range(2)]
    threads = oracle.max_threads()
    states = np.full(B, dfa[2], dtype=np.int32)
    # bounded sample: each "step" of this arm is one whole-batch oracle step
    steps = max(1, min(args.steps, 40))
    warm = max(1, min(args.warmup, 3))
    for i in range(warm):
        oracle.step([dfa], vb, vo, pools[i % 2], states, threads=threads)
    t0 = time.perf_counter()
    for i in range(steps):
        res = oracle.step([dfa], vb, vo, pools[i % 2], states, threads=threads)
        states = np.where(res["states"] < 0, dfa[2], res["states"]).astype(np.int32)
    dt = time.perf_counter() - t0
    value = B * V * steps / dt
    sample = "%d whole-batch oracle steps (%d rows x %d tokens) of %s" % (steps, B, V, WORKLOAD)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": dt / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "vocab": V, "batch": B, "dfa_states": int(dfa[0].shape[0]),
                   "sampler": "greedy", "note": "CPU oracle, host cores only"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2407_08103_b200 import build as libbuild
    from paper_2407_08103_b200 import cstr
    from paper_2407_08103_b200.decode import ConstrainedDecoder, PushdownDecoder
    from synth import normal_logits
    libbuild.build_library()

    if args.download_only:
        from synth.configs import config_vocab
        from synth.constraints import STRING_LITERAL_REGEX
        from synth.regex_frontend import regex_to_dfa
        vb, vo = config_vocab(WORKLOAD)
        dfa = regex_to_dfa(STRING_LITERAL_REGEX.replace("{0,4096}", "{0,2048}"))
        table = cstr.cstr_table_create(cstr.cstr_load_vocab(vb, vo), dfa[0].shape[0])
        cstr.cstr_table_build(table, cstr.cstr_load_dfa(*dfa))
        torch.cuda.synchronize()
        ms = []
        for lo in (0, 1000, 2000, 3000):
            t0 = time.perf_counter()
            nxt, _ = cstr.cstr_table_download(table, lo, lo + 256)
            ms.append((time.perf_counter() - t0) * 1e3)
        print(json.dumps({"table_download": {"states_per_slab": 256, "vocab": vo.size - 1,
                                             "host_ms_per_slab": float(np.mean(ms[1:])),
                                             "logical_bytes_per_slab": int(nxt.nbytes)}}))
        return
    if args.step_only:
        print(json.dumps({"step_variant": time_step_variant(torch, cstr, args.step_only, dev,
                                                            torch.cuda.current_stream())}))
        return
    if args.build_only == "wildcard":
        from synth.configs import config_vocab
        vb, vo = config_vocab("string_256k")
        print(json.dumps({"wildcard_table_build": time_wildcard_build(
            torch, cstr, cstr.cstr_load_vocab(vb, vo), vb, vo, torch.cuda.current_stream(),
            *measured_hbm_peak())}))
        return
    if args.build_only == "small_constraints":
        from synth.configs import config_vocab
        vb, vo = config_vocab("string_256k")
        print(json.dumps({"small_constraint_compiles": time_small_compiles(
            torch, cstr, cstr.cstr_load_vocab(vb, vo), torch.cuda.current_stream())}))
        return
    if args.build_only:
        print(json.dumps({"table_build": time_build_only(torch, cstr, args.build_only, args.case,
                                                         torch.cuda.current_stream(),
                                                         walker=args.walker)}))
        return
    if args.pushdown_only:
        entry = time_pushdown(torch, cstr, PushdownDecoder, dev, torch.cuda.current_stream(),
                              *measured_hbm_peak(), B=128 if args.case == "small" else 512,
                              steps=max(args.steps, 1) if args.steps < 100 else 48)
        print(json.dumps({"pushdown_step": entry}))
        return

    w, dfa, vb, vo = workload_inputs(args.case)
    V = vo.size - 1
    B = w.batch
    S = int(dfa[0].shape[0])
    K, W = args.steps, max(args.warmup, 3)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        return reduce_max(x, world, dev)

    # ---- set-up: vocabulary, DFA, table (the table build is timed below) ----
    torch.zeros(1, device=dev)                     # CUDA context and module load are not the vocabulary's cost
    vocab_load_ms = []
    for _ in range(2):                             # once per LM: sort, descriptors, upload
        t_v0 = time.perf_counter()
        vocab = cstr.cstr_load_vocab(vb, vo)
        vocab_load_ms.append((time.perf_counter() - t_v0) * 1e3)
    vocab_load_ms = min(vocab_load_ms)
    h_dfa = cstr.cstr_load_dfa(*dfa)
    table = cstr.cstr_table_create(vocab, S)
    build_ms = []
    for _ in range(4):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        cstr.cstr_table_build(table, h_dfa, -1, stream)
        e1.record(stream)
        e1.synchronize()
        build_ms.append(e0.elapsed_time(e1))
    dfa_load_ms, build_e2e_ms = [], []
    for _ in range(3):                     # end to end: DFA upload + build, host clock
        t_e2e0 = time.perf_counter()
        h2 = cstr.cstr_load_dfa(*dfa)
        dfa_load_ms.append((time.perf_counter() - t_e2e0) * 1e3)
        cstr.cstr_table_build(table, h2, -1, stream)
        torch.cuda.synchronize()
        build_e2e_ms.append((time.perf_counter() - t_e2e0) * 1e3)
    dfa_load_ms, build_e2e_ms = min(dfa_load_ms), min(build_e2e_ms)

    # ---- inputs: pinned host pool (rows keyed by global row id), device pool ----
    host_pool = [torch.empty((B, V), dtype=torch.float32).pin_memory() for _ in range(POOL)]
    for k in range(POOL):
        normal_logits(w.logits_seed, k, global_rows(rank, B), V, out=host_pool[k].numpy())
    dev_pool = [t.to(dev, non_blocking=True) for t in host_pool]
    out_bufs = [torch.empty((B, V), dtype=torch.float32, device=dev) for _ in range(2)]
    dec = ConstrainedDecoder(table, B, device=dev)
    start_vec = torch.full((B,), int(dfa[2]), dtype=torch.int32, device=dev)
    torch.cuda.synchronize()

    def one_step(i, logits):
        dec.step(logits, masked_out=out_bufs[i & 1], stream=stream)
        # continuous batching: a finished row is replaced by a fresh sequence
        torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)

    sampler = ClockSampler(local_rank)
    sampler.start()

    # ---- device-resident timing ------------------------------------------
    for i in range(W):
        one_step(i, dev_pool[i % POOL])
    dec.status()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_dev0 = time.perf_counter()
    e0.record(stream)
    for i in range(K):
        one_step(i, dev_pool[i % POOL])
    e1.record(stream)
    barrier()
    t_dev1 = time.perf_counter()
    dev_ms = max_over_ranks(e0.elapsed_time(e1))
    bad, empty = dec.status()

    # duration of the step kernel alone (events around each launch; the restart
    # op runs outside the bracket), for the roofline
    ks = min(K, 128)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(ks)]
    for i in range(ks):
        pairs[i][0].record(stream)
        dec.step(dev_pool[i % POOL], masked_out=out_bufs[i & 1], stream=stream)
        pairs[i][1].record(stream)
        torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)
    torch.cuda.synchronize()
    kernel_ms = float(np.mean([a.elapsed_time(b) for a, b in pairs]))
    kernel_ms_best = float(np.min([a.elapsed_time(b) for a, b in pairs]))
    active_frac = float((dec.states >= 0).float().mean().item())
    # a plain copy moving as many bytes as one step launch, timed the same way
    same_copy_ms = time_copy_of(torch, B * V * BYTES_PER_LOGIT_F32_GREEDY, dev, stream)

    # ---- speculative verification: 64 sequences x (7 drafted + 1) positions --------
    # one fused step over the state history (the 512 rows of the workload) + accept / rewind
    spec = None
    if rank == 0 and B % 8 == 0:
        kk, seqs = 7, B // 8
        hist = dec.states.clone()                      # stands for the draft's state history
        t_st = torch.empty(B, dtype=torch.int32, device=dev)
        t_tok = torch.empty(B, dtype=torch.int32, device=dev)
        draft = torch.zeros((seqs, kk), dtype=torch.int32, device=dev)
        n_acc = torch.empty(seqs, dtype=torch.int32, device=dev)
        out_tok = torch.empty((seqs, kk + 1), dtype=torch.int32, device=dev)
        new_st = torch.empty(seqs, dtype=torch.int32, device=dev)
        sp = []
        for i in range(12):
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record(stream)
            cstr.cstr_step_history([table], dev_pool[i % POOL], hist, t_st, t_tok, out_bufs[i & 1],
                                   dec.ws, stream=stream)
            cstr.cstr_accept_draft(draft, t_tok.view(seqs, kk + 1), t_st.view(seqs, kk + 1), n_acc,
                                   out_tok, new_st, stream=stream)
            s1.record(stream)
            s1.synchronize()
            sp.append(s0.elapsed_time(s1))
        spec_ms = float(np.mean(sp[2:]))
        spec = {"sequences": seqs, "drafted_tokens": kk, "rows": B, "ms": spec_ms,
                "logits_per_s": B * V / (spec_ms * 1e-3),
                "roofline": roofline_entry(B * V * BYTES_PER_LOGIT_F32_GREEDY / (spec_ms * 1e-3) / 1e9,
                                           *measured_hbm_peak()),
                "kernels": "step_vec_kernel over the state history + accept_draft_kernel"}

    # ---- end to end: pinned host logits in, results out, every step -------------
    # twice: tokens + states back (what a sampler needs), and with the penalised logits
    # copied back to pinned host memory as well (every result of the step)
    staging = [torch.empty((B, V), dtype=torch.float32, device=dev) for _ in range(2)]
    h_tok = torch.empty(B, dtype=torch.int32).pin_memory()
    h_st = torch.empty(B, dtype=torch.int32).pin_memory()
    h_masked = torch.empty((B, V), dtype=torch.float32).pin_memory()
    Ke = min(K, 64)

    def e2e_step(i, with_masked):
        # one C-ABI call: pinned host logits in (sliced uploads overlapped with the step
        # kernels), tokens + states (+ penalised logits) back on the host when it returns
        cstr.cstr_step_host([table], host_pool[i % POOL], dec.states, h_tok, staging[0], staging[1],
                            dec.tokens, dec.ws, states_host=h_st,
                            masked_host=h_masked if with_masked else None, stream=stream)
        torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)

    e2e_ms = e2e_full_ms = float("nan")
    if not args.skip_e2e:
        for with_masked in (False, True):
            dec.reset()
            for i in range(3):
                e2e_step(i, with_masked)
            barrier()
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(stream)
            for i in range(Ke):
                e2e_step(i, with_masked)
            f1.record(stream)
            barrier()
            if with_masked:
                e2e_full_ms = max_over_ranks(f0.elapsed_time(f1))
            else:
                e2e_ms = max_over_ranks(f0.elapsed_time(f1))

    # ---- the bandwidth-bound bf16 legs: the same table, 512 x 256,000 bf16 logits,
    # greedy and Gumbel-max (device-generated seeded values: timing only)
    bf16_legs = None
    if rank == 0 and args.case == "full" and not args.skip_other_workloads:
        bf16_legs = []
        gen = torch.Generator(device=dev)
        gen.manual_seed(w.logits_seed + 7)
        bpool = [torch.randn((B, V), generator=gen, device=dev).to(torch.bfloat16) for _ in range(POOL)]
        bout = [torch.empty((B, V), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        u = torch.rand((B, V), generator=gen, device=dev).clamp_(1e-20, 1 - 1e-7)
        gnoise = [-torch.log(-torch.log(u)), None]
        u = torch.rand((B, V), generator=gen, device=dev).clamp_(1e-20, 1 - 1e-7)
        gnoise[1] = -torch.log(-torch.log(u))
        del u
        peak_now, kind_now = measured_hbm_peak()
        for gumbel in (False, True):
            dec.reset()
            bp = []
            for i in range(36):
                b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                b0.record(stream)
                dec.step(bpool[i % POOL], noise=gnoise[i & 1] if gumbel else None,
                         masked_out=bout[i & 1], stream=stream)
                b1.record(stream)
                torch.where(dec.states < 0, start_vec, dec.states, out=dec.states)
                if i >= 4:
                    bp.append((b0, b1))
            torch.cuda.synchronize()
            ms = float(np.mean([a.elapsed_time(b) for a, b in bp]))
            bpl = 2 + 2 + (4 if gumbel else 0) + 1.0 / 8.0
            bf16_legs.append({
                "workload": "%s table, batch %d x vocab %d, bf16 logits, %s" %
                            (WORKLOAD, B, V, "gumbel-max (fp32 noise)" if gumbel else "greedy"),
                "kernel": "step_vec_kernel<bf16, %s>" % ("noise" if gumbel else "greedy"),
                "step_kernel_ms": ms, "logits_per_s": B * V / (ms * 1e-3),
                "roofline": roofline_entry(B * V * bpl / (ms * 1e-3) / 1e9, peak_now, kind_now,
                                           bytes_per_logit=bpl,
                                           logits_pool="%d tensors x %.1f MB" % (POOL, B * V * 2 / 1e6))})
        del bpool, bout, gnoise
        torch.cuda.empty_cache()
        dec.reset()
    sampler.stop_flag.set()
    sampler.join(timeout=2)
    clocks = sampler.summary(t_dev0, t_dev1)

    # ---- table-build scaling workload: random 10,000-state DFA ------------
    build_random = None
    if not args.skip_build_bench and rank == 0:
        from synth import random_range_dfa
        n_rd = 10000 if args.case == "full" else 4096
        rd = random_range_dfa(n_rd, seed=2)
        h_rd = cstr.cstr_load_dfa(*rd)
        t_rd = cstr.cstr_table_create(vocab, n_rd)
        ms = []
        for _ in range(4):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            cstr.cstr_table_build(t_rd, h_rd, -1, stream)
            a1.record(stream)
            a1.synchronize()
            ms.append(a0.elapsed_time(a1))
        build_random = ms[1:]
        del t_rd, h_rd

    small = None
    if rank == 0 and world == 1 and not args.skip_other_workloads and args.case == "full":
        small = time_small_batches(torch, cstr, table, V, dev, stream)

    small_compiles = None
    if not args.skip_build_bench and rank == 0 and args.case == "full":
        small_compiles = time_small_compiles(torch, cstr, vocab, stream)

    wildcard = None
    if not args.skip_build_bench and rank == 0 and args.case == "full":
        wildcard = time_wildcard_build(torch, cstr, vocab, vb, vo, stream, *measured_hbm_peak())

    # ---- the other four workloads (single-GPU runs only) --------------------
    others, pushdown = None, None
    if rank == 0 and world == 1 and not args.skip_other_workloads and args.case == "full":
        del dev_pool, staging, out_bufs
        torch.cuda.empty_cache()
        peak_now, kind_now = measured_hbm_peak()
        pushdown = time_pushdown(torch, cstr, PushdownDecoder, dev, stream, peak_now, kind_now)
        torch.cuda.empty_cache()
        others = []
        for name in ("api_1k", "json_32k", "schema40_128k", "random10k_256k"):
            others.append(time_other_workload(name, torch, cstr, ConstrainedDecoder, dev, stream,
                                              peak_now, kind_now))
            torch.cuda.empty_cache()

    # ---- CPU baseline: the oracle on the host cores (rank 0, N = 1) --------
    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        pools = [host_pool[k].numpy() for k in range(2)]
        v, cores, sample, _ = time_oracle(w, dfa, vb, vo, pools, args.cpu_seconds, 400)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
               "cpu_model": cpu_model_string(), "host_threads_available": os.cpu_count(),
               "single_thread_value": time_oracle_single_thread(dfa, vb, vo, pools[0]),
               "table_build": time_oracle_table_build(dfa, vb, vo)}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_hbm_peak()
    logits_per_step = B * V * world
    value = whole_job_throughput(B * V, world, K, dev_ms)
    step_bytes = B * V * BYTES_PER_LOGIT_F32_GREEDY
    achieved = step_bytes / (kernel_ms * 1e-3) / 1e9
    bt = np.array(build_ms[1:])
    transitions = S * V

    def build_entry(ms_list, s_states, workload):
        ms_best = float(np.mean(ms_list))
        tps = s_states * V / (ms_best * 1e-3)
        gbs = s_states * V * BYTES_PER_TRANSITION / (ms_best * 1e-3) / 1e9
        return {"workload": workload, "dfa_states": s_states, "vocab": V, "ms": ms_best,
                "value": tps, "unit": "transitions/s",
                "roofline": roofline_entry(gbs, peak, peak_kind,
                                           note="stores of next (int16) + mask only")}

    e2e = None
    if not args.skip_e2e:
        e2e = {"value": logits_per_step * Ke / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": B * V * 4, "d2h_bytes_per_step": B * 8, "steps": Ke,
               "ms_per_step": e2e_ms / Ke,
               "note": "cstr_step_host per step: pinned host logits -> device in 8 row slices overlapped "
                       "with the step kernels, tokens + states -> host, synchronous; the penalised "
                       "logits stay on the device",
               "with_masked_logits": {
                   "value": logits_per_step * Ke / (e2e_full_ms * 1e-3), "unit": UNIT,
                   "h2d_bytes_per_step": B * V * 4, "d2h_bytes_per_step": B * V * 4 + B * 8,
                   "steps": Ke, "ms_per_step": e2e_full_ms / Ke,
                   "note": "the same call with masked_host given: every result of the step (tokens, "
                           "states and the penalised logits) is in pinned host memory when it returns; "
                           "downloads of earlier slices overlap the uploads of later ones"}}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": dev_ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD if args.case == "full" else WORKLOAD + " (small profiling case)",
                   "vocab": V, "batch": B, "dfa_states": S,
                   "sampler": "greedy", "logits": "fp32 N(0,1), pool of %d seeded tensors" % POOL,
                   "l2": "inputs larger than L2 (each logits tensor %.0f MB, rotated)" % (B * V * 4 / 1e6),
                   "rows": "finished rows restart at the start state (all rows active)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "e2e": e2e,
        "gpu_launches": K,
        "clocks": clocks,
        "roofline": roofline_entry(
            achieved, peak, peak_kind, traffic=step_traffic_bytes(B * V),
            traffic_source="ncu DRAM counters of the small profiling case (128 rows): reads scaled by "
                           "the logits per launch, writes = algorithmic less the output still in L2 at "
                           "the end; null when the kernel source changed since",
            kernel="step_vec_kernel<fp32, greedy>", kernel_ms=kernel_ms,
            kernel_ms_best=kernel_ms_best, launches_timed=ks, bytes_per_launch=step_bytes,
            same_size_copy_ms=same_copy_ms, frac_of_same_size_copy=same_copy_ms / kernel_ms,
            active_row_fraction_at_end=active_frac),
        "inputs_sha256": inputs_sha256(dfa, vb, vo, host_pool[0][0].numpy()),
        "cpu_baseline": cpu,
        "table_build": [build_entry(bt, S, WORKLOAD)] +
                       ([build_entry(build_random, 10000 if args.case == "full" else 4096,
                                     "random10k_256k (DFA 0)" if args.case == "full"
                                     else "random 4,096-state DFA (small profiling case)")]
                        if build_random else []),
        "table_build_e2e_ms": build_e2e_ms,
        "dfa_load_ms": dfa_load_ms,
        "vocab_load_ms": vocab_load_ms,
        "wildcard_table_build": wildcard,
        "small_constraint_compiles": small_compiles,
        "speculative_verify": spec,
        "pushdown_step": pushdown,
        "small_batch_step_latency": small,
        "other_workloads": others,
        "bf16_step_512x256k": bf16_legs,
        "status_rows": {"bad_state": bad, "empty_mask": empty},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
