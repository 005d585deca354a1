#!/usr/bin/env python
"""Benchmark of the lookahead-importance hot path: one step = spec_score -> spec_pool_topk ->
spec_compact_kv (SpecPC workload: spec_score -> specpc_token_select) over ALL layers of one
synthetic workload.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

metric  : prompt tokens scored + compacted per second (all layers), whole job over N GPUs.
value   : device-timed (CUDA events), inputs resident in HBM.
e2e     : same metric with the host->device copy of Q/K/V from pinned memory and the
          device->host read of the selection inside the timed region.
roofline: the scoring call (two tensor-core passes) against the measured burst bf16 peak (the
          fraction of the sustained peak is printed beside it; it becomes `frac` only when the
          run's own clock samples show the power cap inside the timed region).
cpu_baseline: the fp64 oracle timed on the host cores on a bounded sample (rank 0, N = 1).
With N > 1 every rank runs the same per-GPU workload (weak scaling, no data-path collective).
The default workload is the 128K-token one the performance target is stated on; --config picks
another.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "prompt_tokens_scored_and_compacted_per_s_all_layers"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per layer of the workload, from the ncu
# captures summarised under profiles/ (small cases; traffic grows in proportion to the layers), with the
# first 16 hex digits of the SHA-256 of the kernel source the capture was taken on.  A changed source
# makes the figure stale and it is reported as null.
NCU_TRAFFIC = {
    # workload index -> {kernel group: (bytes per layer, source files, hash of those sources)}
    # profiles/score_kernel_c2.md (2 layers) and profiles/select_and_gather_c2.md (8 layers)
    2: {"score": ((542.008064e6 + 7.79392e6 + 550.035456e6 + 11.079168e6) / 2, ["score.cu"], "d44fc0da3556a83b"),
        "select": ((8.407296e6 + 33.585152e6 + 0.004864e6 + 3.372288e6) / 8, ["select_stream.cu", "select_common.cuh"], "44e0bb49c4dfc6e9"),
        "gather": ((67.679488e6 + 13.955328e6) / 8, ["compact.cu"], "4de11f4bd31ee049")},
    # profiles/select_and_gather_c2.md, the capture of all 32 layers of workload 1 (unit_select_kernel, compact_bulk_kernel)
    1: {"select": (16.861952e6 / 32, ["select_stream.cu", "select_common.cuh"], "44e0bb49c4dfc6e9"),
        "gather": ((135.294976e6 + 75.415808e6) / 32, ["compact.cu"], "4de11f4bd31ee049")},
}


def source_digest(files):
    import hashlib
    h = hashlib.sha256()
    for src in files:
        with open(os.path.join(ROOT, "paper_2506_08373_b200", "csrc", src), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(config: int, group: str, n_layers: int):
    ent = NCU_TRAFFIC.get(config, {}).get(group)
    if ent is None:
        return None
    per_layer, files, digest = ent
    try:
        if source_digest(files) != digest:
            return None
    except OSError:
        return None
    return per_layer * n_layers


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "of measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "of fallback"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index (2 = Llama-3.1-8B shape at 128K tokens, the one the target is stated on)")
    ap.add_argument("--layers", type=int, default=0, help="debug/profiling only: run the first LAYERS layers")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    return ap.parse_args(argv)


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's time (the job finishes when the last rank does)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(tokens_per_rank: int, steps: int, world: int, max_ms_total: float) -> float:
    """Whole-job throughput: every rank processed `tokens_per_rank` prompt tokens per step."""
    return world * tokens_per_rank * steps / (max_ms_total * 1e-3)


# ------------------------------------------------------------------ clocks ------------

class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark_begin(self):
        """Wall-clock start of the timed region (the sampler itself starts earlier: nvidia-smi needs a
        few hundred milliseconds before its first sample)."""
        self.t_begin = time.time()

    def stop(self):
        t_end = time.time()
        t_begin = getattr(self, "t_begin", 0.0)
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            time.sleep(0.06)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        try:
            import datetime
            self.file.flush()
            self.file.seek(0)
            rows = []
            for line in self.file.read().strip().splitlines():
                r = [x.strip() for x in line.split(",")]
                if len(r) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                except Exception:
                    ts = None
                rows.append((ts, r[1:]))
            inside = [r for ts, r in rows if ts is not None and t_begin - 0.01 <= ts <= t_end + 0.01]
            if not inside:                                   # clock skew or a very short region: the last samples
                inside = [r for _, r in rows[-3:]]
            sm = [float(r[0]) for r in inside]
            if sm:
                out["sm_mhz"] = statistics.median(sm)
                out["sm_max_mhz"] = float(inside[0][1])
                try:
                    out["power_w"] = statistics.median(float(r[2]) for r in inside)
                except Exception:
                    pass
                out["samples"] = len(sm)
                names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
                for i, n in enumerate(names):
                    if any(r[4 + i].lower().startswith("active") for r in inside):
                        out["reasons"].append(n)
        except Exception:
            pass
        finally:
            try:
                self.file.close()
                os.unlink(self.file.name)
            except Exception:
                pass
        return out


# ------------------------------------------------------------------ workload ----------

class State:
    """Device-resident inputs, outputs and scratch of one workload."""

    def __init__(self, B, W, w, device, layers):
        import torch
        self.B, self.w, self.device = B, w, device
        self.L = len(layers)
        self.q, self.k, self.v = W.gen_layers(w, layers, device, want_v=(w.n_neighbor == 0))
        self.cu = W.cu_seqlens(w)
        self.T = self.cu[-1]
        self.cu_t = torch.tensor(self.cu, dtype=torch.int32, device=device) if w.n_seq > 1 else None
        self.pr = B.make_problem(n_layers=self.L, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                                 head_dim=w.head_dim, n_lookahead=w.n_lookahead, n_window=w.n_window,
                                 softmax_scale=w.scale, total_tokens=self.T,
                                 n_in=(w.n_in if w.n_in is not None else max(W.seq_lens(w))), n_seq=w.n_seq,
                                 cu_seqlens=self.cu_t, k=self.k, v=self.v)
        self.ws = torch.empty(B.spec_workspace_bytes(self.pr), dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.scores = torch.empty((self.L, w.n_kv_heads, self.T), dtype=torch.float32, device=device)
        self.specpc = w.n_neighbor > 0
        self.row_weight, self.pr_keep, self.scores_keep = None, self.pr, self.scores
        if w.paper_specpc:
            # Algorithm 2 lines 2-6: window row j weighs j / n_window, lookahead rows 1; the first l_skip layers
            # stay out of the token scores (pointer offset into the score tensor)
            self.row_weight = torch.cat([torch.arange(1, w.n_window + 1, dtype=torch.float32) / w.n_window,
                                         torch.ones(w.n_lookahead)]).to(device)
            skip = min(w.l_skip, self.L - 1)
            self.scores_keep = self.scores[skip:]
            self.pr_keep = B.make_problem(n_layers=self.L - skip, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                                          head_dim=w.head_dim, n_lookahead=w.n_lookahead, n_window=w.n_window,
                                          softmax_scale=w.scale, total_tokens=self.T, n_in=w.n_in, n_seq=w.n_seq,
                                          cu_seqlens=self.cu_t)
        if self.specpc:
            self.cap = (min(max(W.seq_lens(w)), w.c_max + w.n_window) if w.paper_specpc else
                        min(max(W.seq_lens(w)), w.c_max * (2 * w.n_neighbor + 1)))
            self.keep = torch.empty((w.n_seq, self.cap), dtype=torch.int32, device=device)
            self.n_keep = torch.empty((w.n_seq,), dtype=torch.int32, device=device)
            self.results = [self.keep, self.n_keep]
        else:
            self.idx = torch.empty((w.n_seq, self.L, w.n_kv_heads, w.c_max), dtype=torch.int32, device=device)
            self.cnt = torch.empty((w.n_seq, self.L, w.n_kv_heads), dtype=torch.int32, device=device)
            self.bt = None
            if w.page_size:
                self.bt = W.block_table(w, device)
                self.n_pages = self.bt.numel()
                shape = (self.L, self.n_pages, w.n_kv_heads, w.page_size, w.head_dim)
            else:
                shape = (w.n_seq, self.L, w.n_kv_heads, w.c_max, w.head_dim)
            self.k_out = torch.empty(shape, dtype=torch.bfloat16, device=device)
            self.v_out = torch.empty(shape, dtype=torch.bfloat16, device=device)
            # what the path produces: the index lists and the compacted cache
            self.results = [self.idx, self.cnt, self.k_out, self.v_out]
        # kernels of the library per step: two scoring passes + merge; keep set: reduce + cluster select;
        # else the selection (sample floor + sweep + finish; one kernel for up to 592 units of up to 16384
        # positions, and for a budget above a sixth of the sequence) and the gather
        max_len = w.len_hi if w.n_seq > 1 else w.n_in
        n_units = w.n_seq * self.L * w.n_kv_heads
        self.select_kernels = ("sample_floor + stream_sweep + stream_finish" if w.c_max * 6 <= max_len and
                               (max_len + 3 > 16384 + (3 if w.n_seq == 1 else 0) or n_units > 592) else
                               "unit_select" if w.c_max * 6 <= max_len else "cluster_select")
        self.launches_per_step = 3 + ((3 if w.paper_specpc else 2) if self.specpc else
                                      (3 if self.select_kernels.startswith("sample") else 1) + 1)

    def step(self, events=None, v_src=None):
        B, w = self.B, self.w
        v = self.v if v_src is None else v_src
        if events is not None:
            events[0].record()
        B.spec_score(self.pr, self.q, self.k, self.scores, self.ws, row_weight=self.row_weight,
                     reduce=B.REDUCE_MAX if w.paper_specpc else B.REDUCE_SUM, status_word=self.status)
        if events is not None:
            events[1].record()
        if w.paper_specpc:
            B.specpc_token_select(self.pr_keep, self.scores_keep, B.REDUCE_MAX, B.POOL_AVG_THEN_MAX, w.pool_k, w.c_max,
                                  w.n_neighbor, w.n_window, self.keep, self.cap, self.n_keep, self.ws, status_word=self.status)
            if events is not None:
                events[2].record()
                events[3].record()
        elif self.specpc:
            B.specpc_token_select(self.pr, self.scores, B.REDUCE_SUM, B.POOL_MAX, w.pool_k, w.c_max, w.n_neighbor, 0,
                                  self.keep, self.cap, self.n_keep, self.ws, status_word=self.status)
            if events is not None:
                events[2].record()
                events[3].record()
        else:
            B.spec_pool_topk(self.pr, self.scores, B.POOL_MAX, w.pool_k, w.c_max, 0, self.idx, self.cnt,
                             workspace=self.ws, status_word=self.status)
            if events is not None:
                events[2].record()
            if self.bt is not None:
                B.spec_compact_kv(self.pr, self.k, v, self.idx, w.c_max, self.k_out, self.v_out,
                                  block_table=self.bt, page_size=w.page_size, n_pages=self.n_pages,
                                  status_word=self.status)
            else:
                B.spec_compact_kv(self.pr, self.k, v, self.idx, w.c_max, self.k_out, self.v_out,
                                  status_word=self.status)
            if events is not None:
                events[3].record()


def algorithmic_work(w, L, tokens):
    """Algorithmic flops and bytes of one step (the per-unit figures times the units of a launch)."""
    R, d, C = w.rows, w.head_dim, w.c_max
    flops_one_pass = 2.0 * L * w.n_q_heads * R * tokens * d
    k_bytes_one_pass = 2.0 * d * w.n_kv_heads * L * tokens
    score_bytes = 4.0 * w.n_kv_heads * L * tokens
    select_bytes = score_bytes + 4.0 * w.n_kv_heads * L * C * w.n_seq
    gather_bytes = 0.0 if w.n_neighbor else 8.0 * w.n_kv_heads * L * C * d * w.n_seq
    return {"flops_two_pass": 2 * flops_one_pass, "flops_one_pass": flops_one_pass,
            "score_hbm_bytes": 2 * k_bytes_one_pass + score_bytes, "select_bytes": select_bytes,
            "gather_bytes": gather_bytes}


class OracleSample:
    """A bounded sample of the workload for the CPU oracle: the first `n_layers` layers, all sequences
    and KV heads, generated once on the host."""

    def __init__(self, W, w, n_layers):
        import numpy as np
        import torch
        import oracle
        oracle.build()
        self.oracle, self.w = oracle, w
        bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
        self.layers = list(range(min(n_layers, w.n_layers)))
        q, k, v = W.gen_layers(w, self.layers, "cpu", want_v=(w.n_neighbor == 0))
        self.cu = W.cu_seqlens(w)
        self.qb, self.kb = bits(q), bits(k)
        self.vb = bits(v) if v is not None else None

    def run(self):
        """One pass of the whole path over the sample; seconds of wall time."""
        o, w = self.oracle, self.w
        t0 = time.perf_counter()
        if w.paper_specpc:
            import numpy as np
            rw = np.concatenate([np.arange(1, w.n_window + 1) / w.n_window, np.ones(w.n_lookahead)])
            sc = o.spec_score(self.qb, self.kb, self.cu, w.n_lookahead, w.n_window, w.scale, row_weight=rw, mode=o.MAX)
        else:
            sc = o.spec_score(self.qb, self.kb, self.cu, w.n_lookahead, w.n_window, w.scale)
        if w.paper_specpc:
            o.specpc_select(sc[min(w.l_skip, len(self.layers) - 1):], self.cu, o.MAX, o.POOL_AVG_THEN_MAX, w.pool_k, w.c_max,
                            w.n_neighbor, w.n_window)
        elif w.n_neighbor:
            o.specpc_select(sc, self.cu, o.SUM, o.POOL_MAX, w.pool_k, w.c_max, w.n_neighbor, 0)
        else:
            idx, _, _, _ = o.pool_topk(sc, self.cu, o.POOL_MAX, w.pool_k, w.c_max)
            o.compact(self.kb, self.cu, idx)
            o.compact(self.vb, self.cu, idx)
        return time.perf_counter() - t0

    def describe(self, dt):
        return ("%d of %d layers, all sequences and KV heads (%d independent units over %d threads), %.1f s wall; "
                "scaled by layers" % (len(self.layers), self.w.n_layers,
                                      len(self.layers) * self.w.n_seq * self.w.n_kv_heads, self.oracle.threads(), dt))

    def value(self, dt):
        return self.cu[-1] / (dt * self.w.n_layers / len(self.layers))


def layers_filling_the_cores(w):
    """Fewest layers whose (sequence, KV head) units keep every oracle thread busy."""
    import oracle
    oracle.build()
    per_layer = w.n_seq * w.n_kv_heads
    return max(1, min(w.n_layers, -(-oracle.threads() // per_layer)))


def cpu_baseline(W, w, seconds=12.0):
    """The oracle, as it stands, on a bounded sample of about `seconds` of work."""
    base = layers_filling_the_cores(w)
    sample = OracleSample(W, w, base)
    dt = sample.run()
    more = int(min(w.n_layers // base, max(1, seconds / max(dt, 1e-3)))) * base
    if more > base:
        sample = OracleSample(W, w, more)
        dt = sample.run()
    return {"value": sample.value(dt), "unit": UNIT, "cores": sample.oracle.threads(), "kind": "oracle",
            "sample": sample.describe(dt)}


def config_dict(w, n_layers, tokens, kv_bytes, world, note=""):
    return {"workload": w.name + note, "n_layers": n_layers, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "tokens_per_step": tokens, "n_seq": w.n_seq, "n_lookahead": w.n_lookahead,
            "n_window": w.n_window, "pool_k": w.pool_k, "c_max": w.c_max,
            "l2": "inputs larger than L2 (K+V %.2f GB per step)" % (kv_bytes / 1e9),
            "parallelism": "replicated per GPU, no collective" if world > 1 else "single GPU"}


def run_reference(args, W, w):
    """Reference arm: the CPU oracle, as it stands, on the host cores.  A step is one pass of the whole path
    over a bounded sample (the fewest layers that keep every core busy); the value is scaled to all layers.
    The run stops early, and says so in `steps`, once the timed steps have taken 200 s."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    sample = OracleSample(W, w, layers_filling_the_cores(w))
    times = []
    t_begin = time.perf_counter()
    for i in range(args.warmup + args.steps):
        if i >= 1 and time.perf_counter() - t_begin > 200 and times:
            break
        dt = sample.run()
        if i >= args.warmup or time.perf_counter() - t_begin > 120:   # a slow host: later warm-up steps are counted
            times.append(dt)
    steps = len(times)
    dt = sum(times) / steps
    value = sample.value(dt)
    tokens = sample.cu[-1]
    kv_bytes = (1 if w.n_neighbor else 2) * 2.0 * w.head_dim * w.n_kv_heads * w.n_layers * tokens
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, max(0, args.warmup + args.steps - steps)),
            "ms_per_step": 1e3 * dt * w.n_layers / len(sample.layers), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, w.n_layers, tokens, kv_bytes, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": sample.oracle.threads(), "kind": "oracle",
                             "sample": "each step: " + sample.describe(dt)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main(argv=None):
    args = parse_args(argv)
    from paper_2506_08373_b200 import workloads as W
    w = W.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, W, w)
        return 0

    import torch
    from paper_2506_08373_b200 import binding as B
    B.lib()                                            # fails loudly when the CUDA library is missing
    rank, world, local = dist_env()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    layers = list(range(args.layers if args.layers else w.n_layers))
    st = State(B, W, w, device, layers)
    tokens = st.T
    K, Wm = args.steps, max(args.warmup, 3) if not args.layers else args.warmup

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(Wm):
        st.step()
    torch.cuda.synchronize()
    assert st.status.item() == 0, "device-side error status %d" % st.status.item()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    end = torch.cuda.Event(enable_timing=True)
    if world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark_begin()
    for i in range(K):
        st.step(ev[i])
    end.record()
    torch.cuda.synchronize()
    total_ms = ev[0][0].elapsed_time(end)
    if world > 1:
        torch.distributed.barrier()
    clocks = sampler.stop() if sampler else None
    total_ms = max_over_ranks(total_ms, device)
    assert st.status.item() == 0
    t_score = sum(e[0].elapsed_time(e[1]) for e in ev) / K
    t_select = sum(e[1].elapsed_time(e[2]) for e in ev) / K
    t_gather = sum(e[2].elapsed_time(e[3]) for e in ev) / K

    peaks, peak_src = load_peaks()
    work = algorithmic_work(w, st.L, tokens)
    tf = work["flops_two_pass"] / (t_score * 1e-3) / 1e12
    # The scoring call is compared with the measured burst bf16 peak.  Only when this run's own clock samples
    # show the power cap inside the timed region is the sustained peak (itself measured under the cap) the
    # denominator of `frac`; both fractions are always in the line.
    capped = clocks is not None and "sw_power_cap" in clocks.get("reasons", [])
    peak_tf = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": "spec_score: score_kernel<1> + merge + score_kernel<2>",
                "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf,
                "peak_source": peak_src + (" (sustained cuBLAS bf16: sw_power_cap seen in the timed region)" if capped
                                           else " (burst cuBLAS bf16)"),
                "frac_of_burst_peak": tf / peaks["bf16_tflops"], "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"],
                "frac_of_nominal_dense_bf16_2250": tf / 2250.0,
                "work": "two tensor-core passes (statistics, then probabilities); one contraction is half of it",
                "achieved_one_contraction": tf / 2, "ms": t_score,
                "ms_times_sm_mhz": (t_score * clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
                "algorithmic_bytes": work["score_hbm_bytes"], "traffic": ncu_traffic(args.config, "score", st.L)}
    hbm_bytes = work["select_bytes"] + work["gather_bytes"]
    gbs = hbm_bytes / ((t_select + t_gather) * 1e-3) / 1e9
    roofline_hbm = {"bound": "hbm", "kernel": (st.select_kernels + " + compact_bulk" if not st.specpc
                                                 else "token_reduce + cluster_select"),
                    "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                    "peak_source": peak_src + " (copy)", "ms_select": t_select, "ms_gather": t_gather,
                    "gather_gbs": (work["gather_bytes"] / (t_gather * 1e-3) / 1e9) if t_gather > 0 and work["gather_bytes"] else None,
                    "algorithmic_bytes": hbm_bytes,
                    "traffic_note": "DRAM bytes under ncu on a small case, scaled by layers; gathered rows still in L2 when the "
                                    "capture ended are not in it",
                    "traffic": (None if st.specpc or ncu_traffic(args.config, "select", st.L) is None or ncu_traffic(args.config, "gather", st.L) is None
                                else ncu_traffic(args.config, "select", st.L) + ncu_traffic(args.config, "gather", st.L))}

    line = {"metric": METRIC, "value": job_value(tokens, K, world, total_ms), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": Wm, "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_dict(w, st.L, tokens, (2 if st.v is not None else 1) * st.k.numel() * 2, world,
                                  "" if not args.layers else " (first %d layers only: NOT the quoted configuration)" % args.layers),
            "roofline": roofline, "roofline_hbm": roofline_hbm, "gpu_launches": st.launches_per_step * K,
            "clocks": clocks}

    if rank == 0 and world == 1 and not args.no_e2e:
        line["e2e"] = run_e2e(st, tokens, min(K, 5))
    if rank == 0 and world == 1 and not args.no_cpu:
        del st                                          # the oracle sample needs host memory, not the device
        line["cpu_baseline"] = cpu_baseline(W, w)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


def pinned_like(t, n_layers=None):
    import torch
    shape = list(t.shape)
    if n_layers is not None:
        shape[0] = n_layers
    return torch.empty(shape, dtype=t.dtype, pin_memory=True)


def run_e2e(st, tokens, steps):
    """Host buffers in, product out: every step copies Q/K/V from pinned host memory to the device, runs
    the calls and copies what the path produces (index lists and counts, and the compacted K/V cache; for
    the SpecPC workload the keep list) back to pinned host memory, all inside the timed region."""
    import torch
    dev_in = [t for t in (st.q, st.k, st.v) if t is not None]
    staged_layers = st.L
    while True:
        try:
            host_in = [pinned_like(dev_in[0])] + [pinned_like(t, staged_layers) for t in dev_in[1:]]
            break
        except RuntimeError:                              # not enough page-locked memory: stage fewer layers at a time
            host_in = None
            if staged_layers == 1:
                raise
            staged_layers = (staged_layers + 1) // 2
    host_in[0].copy_(dev_in[0])
    for h, d in zip(host_in[1:], dev_in[1:]):
        h.copy_(d[:staged_layers])
    host_out = [pinned_like(t) for t in st.results]
    torch.cuda.synchronize()

    def copy_in(tensors):
        for h, d in tensors:
            if h.shape[0] == d.shape[0]:
                d.copy_(h, non_blocking=True)
            else:                                         # K / V staged in layer chunks: the same bytes cross the bus
                for l0 in range(0, d.shape[0], staged_layers):
                    c = min(staged_layers, d.shape[0] - l0)
                    d[l0:l0 + c].copy_(h[:c], non_blocking=True)

    def one():
        copy_in(list(zip(host_in, dev_in)))
        st.step()
        for h, d in zip(host_out, st.results):
            h.copy_(d, non_blocking=True)

    one()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    out = {"value": tokens / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": steps,
           "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in dev_in),
           "d2h_bytes_per_step": sum(t.numel() * t.element_size() for t in st.results),
           "moves": "in: Q, K, V; out: " + ("keep list and its length" if st.specpc else
                                             "index lists, counts and the compacted K/V cache"),
           "pinned_staging_layers": staged_layers}
    if st.v is not None and staged_layers == st.L:
        # The same step with V left in pinned host memory: scoring needs Q and K only, and the gather reads
        # the selected V rows straight from the host buffer, so most of V never crosses the bus.
        v_host = host_in[2]
        rows = st.idx.numel() * st.w.head_dim * 2

        def one_v_in_place():
            copy_in(list(zip(host_in[:2], dev_in[:2])))
            st.step(v_src=v_host)
            for h, d in zip(host_out, st.results):
                h.copy_(d, non_blocking=True)

        one_v_in_place()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            one_v_in_place()
        e1.record()
        torch.cuda.synchronize()
        ms2 = e0.elapsed_time(e1) / steps
        out["v_read_in_place"] = {"value": tokens / (ms2 * 1e-3), "unit": UNIT, "ms_per_step": ms2,
                                  "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in dev_in[:2]) + rows,
                                  "note": "V stays in pinned host memory; the gather reads the selected rows over the bus"}
    return out


if __name__ == "__main__":
    sys.exit(main())
