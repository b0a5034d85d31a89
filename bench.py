#!/usr/bin/env python
"""Benchmark of the post-prefill KV-compression pass.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
                    [--rank-mode position|score] [--impl ours|reference]

One step = the fused pass (score, select, compact) over every layer of one
synthetic prefill cache that is already resident in HBM, through one
refree_compress_layers call (layers software-pipelined inside the library); the
time of one refree_compress_layer call per layer is reported beside it.
Prints ONE JSON line on rank 0.  With N > 1 (launched by torchrun) every rank
runs its own replica of the workload: the units of the pass are independent, so
there is no collective on the data path (weak scaling).

`--impl reference` times the CPU oracle on the host cores instead (a bounded
sample of the same workload per step); it exists to put a number beside the
GPU's, not as a target.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "kv_tokens_compressed_per_sec_per_layer"
UNIT = "tokens/s/layer"
DEFAULT_WORKLOAD = "mistral7b_32k"      # the 32K-token, 32q/8kv, d=128 cache the target is quoted on
FALLBACK_HBM_GBS = 6650.0


def log(*a):
    print(*a, file=sys.stderr, flush=True)


# ----------------------------------------------------------- distributed ----
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), \
        int(os.environ.get("WORLD_SIZE", "1"))


def dist_setup(backend: str):
    """Join the process group when launched with WORLD_SIZE > 1."""
    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def dist_barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def dist_max(value: float, world: int, device) -> float:
    """Max over ranks of a host float (the job time is the slowest rank's)."""
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def dist_sum(value: float, world: int, device) -> float:
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def aggregate_throughput(tokens_per_rank: float, ms_per_step_max: float, layers: int, world_tokens: float) -> float:
    """Whole-job tokens/s per layer: tokens all ranks processed in a layer pass / slowest rank's layer time."""
    del tokens_per_rank
    return world_tokens / (ms_per_step_max * 1e-3 / layers)


# ------------------------------------------------------------- clocks ----
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False).name
        self.proc = None
        self.gpu = gpu_index
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu=timestamp,{self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        import datetime
        rows = []
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), parts[4:8]))
            except ValueError:
                continue
        os.unlink(self.path)
        inside = [r for r in rows if self.t0 is not None and self.t0 - 0.05 <= r[0] <= self.t1 + 0.05]
        use = inside if inside else rows[-3:]
        if not use:
            return out
        out["sm_mhz"] = statistics.median(r[1] for r in use)
        out["sm_max_mhz"] = use[0][2]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        out["reasons"] = [n for i, n in enumerate(names) if any(r[3][i].lower().startswith("active") for r in use)]
        out["samples"] = len(inside)
        return out


# ------------------------------------------------------------ workload ----
def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(cfg, seq_lens, lengths):
    """Bytes the pass must move for one layer: K read once for scoring, kept V
    read, kept K and V written, fp32 scores written (the kept-K re-read is
    assumed served from L2).  Returns (1+3rho) form and the (1+4rho) form."""
    row = cfg.head_dim * cfg.elem_bytes
    a = b4 = 0
    for s, n in enumerate(seq_lens):
        for g in range(cfg.num_kv_heads):
            kept = int(lengths[s][g])
            a += n * row + 3 * kept * row + 4 * n
            b4 += n * row + 4 * kept * row + 4 * n
    return a, b4


# dram__bytes_read + dram__bytes_write of one launch of the dominant kernel, from the ncu capture summarised under
# profiles/.  The figure belongs to one version of the kernel source: it is reported only while the source file
# still has the hash it was captured on, and null afterwards.
NCU_TRAFFIC = {
    # workload: (kernel source, first 16 hex digits of its sha256, bytes per launch)
    "mistral7b_32k": ("paper_2502_16886_b200/csrc/score_tc.cu", "848012eefce12c48", 262_343_936 + 92_841_216),
}


def ncu_traffic(cfg, stage):
    import hashlib
    rec = NCU_TRAFFIC.get(cfg.name)
    if stage != "score" or cfg.window != 64 or rec is None:
        return None
    src, digest, nbytes = rec
    try:
        have = hashlib.sha256(open(os.path.join(ROOT, src), "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    return nbytes if have == digest else None


def run_ours(args):
    from paper_2502_16886_b200 import binding, build, workloads
    rank, local_rank, world = dist_setup("nccl")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    build.build()
    binding.lib()
    cfg = workloads.get_config(args.workload)
    if args.window:
        import dataclasses
        cfg = dataclasses.replace(cfg, window=args.window)      # e.g. 1: the paper's default reduced attention
    L = args.layers or cfg.num_layers
    rank_mode = binding.RANK_SCORE if args.rank_mode == "score" else binding.RANK_POSITION
    seq_lens = workloads.sequence_lengths(cfg)
    total = sum(seq_lens)
    cap = cfg.num_kv_heads * total
    units = len(seq_lens) * cfg.num_kv_heads

    t0 = time.time()
    layers = []
    params = None
    for l in range(L):
        lay = workloads.make_layer(cfg, l)
        if params is None:
            params = binding.params_for(cfg, lay, rank_mode=rank_mode, threshold=args.threshold)
        layers.append(dict(
            q=lay.q_win.to(dev), k=lay.k.to(dev), v=lay.v.to(dev),
            k_out=torch.empty(cap, cfg.head_dim, dtype=cfg.torch_dtype, device=dev),
            v_out=torch.empty(cap, cfg.head_dim, dtype=cfg.torch_dtype, device=dev),
            lengths=torch.zeros(units, dtype=torch.int32, device=dev),
            offsets=torch.zeros(units + 1, dtype=torch.int64, device=dev)))
        if l == 0:
            host0 = lay
    seq_start = host0.seq_start.to(dev)
    seq_len = host0.seq_len.to(dev)
    ws = torch.empty(binding.refree_workspace_size(params, total), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if rank == 0:
        log(f"[bench] {cfg.name}: {L} layers generated in {time.time() - t0:.1f}s, "
            f"{torch.cuda.memory_allocated(dev) / 2**30:.1f} GiB on device")

    def one_layer(d):
        binding.refree_compress_layer(params, d["q"], d["k"], d["v"], seq_start, seq_len, total, d["k_out"],
                                      d["v_out"], cap, d["lengths"], d["offsets"], None, None, ws, status)

    def step_per_layer_calls():
        for d in layers:
            one_layer(d)

    # the step: one call for the run of layers (compaction of layer l under the scoring of layer l + 1)
    ptrs = binding.LayerPointers(*[[d[key] for d in layers] for key in ("q", "k", "v", "k_out", "v_out", "lengths", "offsets")])
    ws2 = torch.empty(binding.refree_layers_workspace_size(params, total), dtype=torch.uint8, device=dev)

    def step():
        binding.refree_compress_layers(params, ptrs, seq_start, seq_len, total, cap, ws2, status)

    if args.per_layer_calls:
        step = step_per_layer_calls

    def timed(fn, n):
        dist_barrier(world)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    for _ in range(max(args.warmup, 3)):
        step_per_layer_calls()
    ms_per_layer_calls = timed(step_per_layer_calls, max(3, min(args.steps, 20)))
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = binding.refree_kernel_launch_count()
    sampler.mark_begin()
    # blocks of exactly `steps` steps, each bracketed by barrier + synchronize and timed with CUDA events; repeated
    # until a second of device time has gone by (so the clock sampler sees the load), the median block is reported
    block_ms, spent = [], 0.0
    while not block_ms or (spent < 1000.0 and len(block_ms) < 64):
        block_ms.append(timed(step, args.steps))
        spent += block_ms[-1] * args.steps
        if world > 1:
            spent = dist_max(spent, world, dev)      # every rank runs the same number of blocks
    ms_local = statistics.median(block_ms)
    sampler.mark_end()
    dist_barrier(world)
    launches = (binding.refree_kernel_launch_count() - launches0) // len(block_ms)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = dist_max(ms_local, world, dev)
    ms_per_layer_calls = dist_max(ms_per_layer_calls, world, dev)
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    value = aggregate_throughput(total, ms_step, L, dist_sum(float(total), world, dev))

    if rank != 0:
        if world > 1:
            dist_barrier(world)
        return

    # kept ratio and algorithmic bytes, from the budgets the timed steps produced
    all_lengths = [d["lengths"].view(len(seq_lens), cfg.num_kv_heads).cpu().tolist() for d in layers]
    rho = sum(sum(map(sum, ln)) for ln in all_lengths) / (L * cfg.num_kv_heads * total)
    bytes3 = sum(algorithmic_bytes(cfg, seq_lens, ln)[0] for ln in all_lengths) / L
    bytes4 = sum(algorithmic_bytes(cfg, seq_lens, ln)[1] for ln in all_lengths) / L
    peak, peak_kind = hbm_peak()
    ms_layer = ms_step / L
    pass_gbs = bytes3 / (ms_layer * 1e-3) / 1e9

    # per-stage device times: each stage entry point called back to back over the layers (no synchronisation
    # inside the bracket, so the GPU never idles waiting for a launch), CUDA events around the sweep
    scores = torch.empty(cfg.num_kv_heads, total, dtype=torch.float32, device=dev)
    kept = torch.empty(cap, dtype=torch.int32, device=dev)
    binding.refree_select_budget(params, scores.zero_(), seq_len, total, layers[0]["lengths"], layers[0]["offsets"],
                                 kept, cap, ws, status)
    stage_calls = {
        "score": lambda d: binding.refree_score(params, d["q"], d["k"], seq_start, seq_len, total, scores, ws, status),
        "select": lambda d: binding.refree_select_budget(params, scores, seq_len, total, d["lengths"], d["offsets"],
                                                         kept, cap, ws, status),
        "compact": lambda d: binding.refree_compact(params, d["k"], d["v"], seq_start, seq_len, d["lengths"],
                                                    d["offsets"], kept, d["k_out"], d["v_out"], cap, status),
    }
    stage_ms = {}
    reps = 5
    one_layer(layers[-1])                      # leaves real scores behind for the select sweep
    binding.refree_score(params, layers[-1]["q"], layers[-1]["k"], seq_start, seq_len, total, scores, ws, status)
    for name, call in stage_calls.items():
        for d in layers:
            call(d)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for d in layers:
                call(d)
        e1.record()
        torch.cuda.synchronize()
        stage_ms[name] = e0.elapsed_time(e1) / (reps * L)
    row = cfg.head_dim * cfg.elem_bytes
    kept_rows = rho * cfg.num_kv_heads * total
    stage_bytes = {"score": cfg.num_kv_heads * total * (row + 4), "select": cfg.num_kv_heads * total * 8,
                   "compact": 4 * kept_rows * row + 4 * kept_rows}
    dominant = max(stage_ms, key=stage_ms.get)
    fused_run = (rank_mode == binding.RANK_POSITION and not args.per_layer_calls and cfg.dtype == "bf16"
                 and cfg.head_dim == 128 and 32 <= cfg.group * cfg.window <= 256 and L >= 4)
    if fused_run:
        # The timed step is a chain of L + 1 launches of one kernel (each finishes the scoring of one layer, begins the
        # next and moves the kept rows of the one before: one layer's worth of the whole pass) plus one compaction
        # launch.  Its launch duration is taken live as the marginal time of a layer: a run over all layers against a
        # run over half of them, CUDA events on the stream the call is given.
        half = binding.LayerPointers(*[[d[key] for d in layers[: L // 2]] for key in
                                       ("q", "k", "v", "k_out", "v_out", "lengths", "offsets")])

        def half_step():
            binding.refree_compress_layers(params, half, seq_start, seq_len, total, cap, ws2, status)
        for _ in range(3):
            half_step()
        t_half = statistics.median(timed(half_step, args.steps) for _ in range(5))
        t_full = statistics.median(timed(step, args.steps) for _ in range(5))
        ms_launch = (t_full - t_half) / (L - L // 2)
        dom_gbs = bytes3 / (ms_launch * 1e-3) / 1e9
        roofline = {"kernel": "score_tc_kernel<4>: column pass of layer l - 1, row pass of layer l, kept rows of layer "
                              "l - 2 moved by a warp of the same CTAs (one launch per layer of the timed step)",
                    "bound": "hbm", "achieved": round(dom_gbs, 1), "peak": peak, "peak_kind": f"of {peak_kind}",
                    "unit": "GB/s", "frac": round(dom_gbs / peak, 4), "traffic": ncu_traffic(cfg, "score"),
                    "bytes_per_launch": int(bytes3), "ms_per_launch": round(ms_launch, 5),
                    "how": "marginal time per layer of refree_compress_layers (all layers against half of them)"}
    else:
        dom_gbs = stage_bytes[dominant] / (stage_ms[dominant] * 1e-3) / 1e9
        roofline = {"kernel": f"refree_{dominant} stage", "bound": "hbm", "achieved": round(dom_gbs, 1),
                    "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": round(dom_gbs / peak, 4),
                    "traffic": None, "bytes_per_launch": int(stage_bytes[dominant]),
                    "ms_per_launch": round(stage_ms[dominant], 5)}
    roofline["stages_ms"] = {k: round(v, 5) for k, v in stage_ms.items()}
    roofline["stages_gbs"] = {k: round(stage_bytes[k] / (stage_ms[k] * 1e-3) / 1e9, 1) for k in stage_ms}
    if cfg.window > 1 and cfg.dtype == "bf16" and cfg.head_dim == 128:
        # the scoring stage's three roofs (it forms the logits twice): K once from HBM, the dense contraction
        # at the measured bf16 GEMM rate, one exponential per logit at 16 per clock per SM
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        tf_peak = float(peaks.get("bf16_tflops", 1590.0))
        sm_hz = float(peaks.get("sm_max_mhz", 1965.0)) * 1e6
        logits = 2.0 * cfg.num_kv_heads * total * cfg.group * cfg.window          # both passes
        t_hbm = stage_bytes["score"] / (peak * 1e9) * 1e6
        t_mma = logits * 2 * cfg.head_dim / (tf_peak * 1e12) * 1e6
        t_exp = logits / (148 * 16 * sm_hz) * 1e6
        bound_us = max(t_hbm, t_mma, t_exp)
        roofline["score_stage_roofs"] = {
            "us": {"hbm": round(t_hbm, 2), "tensor": round(t_mma, 2), "exp": round(t_exp, 2)},
            "binding": max((("hbm", t_hbm), ("tensor", t_mma), ("exp", t_exp)), key=lambda kv: kv[1])[0],
            "frac_of_binding": round(bound_us / (stage_ms["score"] * 1e3), 4),
            "tensor_tflops": round(logits * 2 * cfg.head_dim / (stage_ms["score"] * 1e-3) / 1e12, 1),
            "tensor_peak_tflops": tf_peak}
    roofline_pass = {"bound": "hbm", "achieved": round(pass_gbs, 1), "peak": peak, "peak_kind": f"of {peak_kind}",
                     "unit": "GB/s", "frac": round(pass_gbs / peak, 4), "frac_of_8TBps": round(pass_gbs / 8000.0, 4),
                     "bytes_per_layer": int(bytes3), "bytes_per_layer_with_kept_k_reread": int(bytes4),
                     "kept_ratio": round(rho, 4), "ms_per_layer": round(ms_layer, 5),
                     "entry": "refree_compress_layer per layer" if args.per_layer_calls else
                              "refree_compress_layers (one call per step, layers software-pipelined)",
                     "one_call_per_layer": {"ms_per_layer": round(ms_per_layer_calls / L, 5),
                                            "achieved": round(bytes3 / (ms_per_layer_calls / L * 1e-3) / 1e9, 1),
                                            "frac": round(bytes3 / (ms_per_layer_calls / L * 1e-3) / 1e9 / peak, 4)}}

    # the consumer of the pass: one decode step of attention over every layer's compacted cache, swept like a stage
    max_rows = max(seq_lens)
    dws = torch.empty(binding.refree_decode_workspace_size(params, max_rows), dtype=torch.uint8, device=dev)
    q_new = workloads.make_decode_query(cfg, 0, host0.q_win).to(dev)
    dout = torch.empty(len(seq_lens), cfg.num_q_heads, cfg.head_dim, dtype=torch.float32, device=dev)

    def decode(d):
        binding.refree_decode_attention(params, q_new, d["k_out"], d["v_out"], d["offsets"], max_rows, dout, dws, status)

    for d in layers:
        decode(d)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        for d in layers:
            decode(d)
    e1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    dec_ms = e0.elapsed_time(e1) / (reps * L)
    dec_bytes = 2 * kept_rows * row
    dec_gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
    decode_line = {"kernel": "refree_decode_attention", "bound": "hbm", "ms_per_layer": round(dec_ms, 5),
                   "bytes_per_layer": int(dec_bytes), "achieved": round(dec_gbs, 1), "peak": peak,
                   "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": round(dec_gbs / peak, 4)}

    # in-place form of the compaction stage; it overwrites the synthetic cache, so it runs after every other
    # device sweep (a repeat moves the same rows again: same budgets, same traffic)
    def inplace_line_for(anchor, name, bytes_layer):
        def call(d):
            binding.refree_compact_inplace(params, d["k"], d["v"], seq_start, seq_len, d["offsets"], None, status,
                                           anchor=anchor)
        for d in layers:
            call(d)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for d in layers:
                call(d)
        e1.record()
        torch.cuda.synchronize()
        assert int(status.item()) == 0, f"device status {int(status.item())}"
        ms = e0.elapsed_time(e1) / (reps * L)
        gbs = bytes_layer / (ms * 1e-3) / 1e9
        return {"kernel": f"refree_compact_inplace, {name}", "bound": "hbm", "ms_per_layer": round(ms, 5),
                "bytes_per_layer": int(bytes_layer), "achieved": round(gbs, 1), "peak": peak,
                "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": round(gbs / peak, 4)}

    def fused_inplace_ms():
        """The whole pass with end-anchored in-place compaction, one call per layer (overwrites the cache)."""
        ln, of = layers[0]["lengths"], layers[0]["offsets"]

        def call(d):
            binding.refree_compress_layer_inplace(params, d["q"], d["k"], d["v"], seq_start, seq_len, total, ln, of,
                                                  binding.ANCHOR_BACK, ws, status)
        for d in layers:
            call(d)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for d in layers:
                call(d)
        e1.record()
        torch.cuda.synchronize()
        assert int(status.item()) == 0, f"device status {int(status.item())}"
        return e0.elapsed_time(e1) / (reps * L)

    if rank_mode == binding.RANK_POSITION:
        lifted_rows = units * min(cfg.sink, min(seq_lens))
        inplace_line = [
            inplace_line_for(binding.ANCHOR_BACK, "anchored at the end (only the leading rows move)",
                             4 * lifted_rows * row),
            inplace_line_for(binding.ANCHOR_FRONT, "anchored at the front (every kept row moves)",
                             stage_bytes["compact"])]
        fms = fused_inplace_ms()
        inplace_line.append({"kernel": "refree_compress_layer_inplace, anchored at the end (whole pass per layer)",
                             "ms_per_layer": round(fms, 5), "tokens_per_s_per_layer": round(total / (fms * 1e-3), 1)})
    else:
        inplace_line = None

    # the same step in the paper's other settings, on the same device-resident cache: ranking by score (Section 4.4)
    # and the default single query row (Section 3.2 "Reducing Overhead"; the window's last row of every head)
    def variant_record(p_var, qs):
        pv = binding.LayerPointers(qs, *[[d[key] for d in layers] for key in ("k", "v", "k_out", "v_out", "lengths", "offsets")])
        wsv = torch.empty(binding.refree_layers_workspace_size(p_var, total), dtype=torch.uint8, device=dev)

        def run():
            binding.refree_compress_layers(p_var, pv, seq_start, seq_len, total, cap, wsv, status)
        for _ in range(3):
            run()
        ms = statistics.median(timed(run, 5) for _ in range(3)) / L
        assert int(status.item()) == 0, f"device status {int(status.item())}"
        ln = [d["lengths"].view(len(seq_lens), cfg.num_kv_heads).cpu().tolist() for d in layers]
        b3 = sum(algorithmic_bytes(cfg, seq_lens, x)[0] for x in ln) / L
        r = sum(sum(map(sum, x)) for x in ln) / (L * cfg.num_kv_heads * total)
        return {"us_per_layer": round(ms * 1e3, 2), "tokens_per_s_per_layer": round(total / (ms * 1e-3), 1),
                "kept_ratio": round(r, 4), "achieved": round(b3 / (ms * 1e-3) / 1e9, 1), "unit": "GB/s",
                "frac": round(b3 / (ms * 1e-3) / 1e9 / peak, 4), "peak_kind": f"of {peak_kind}"}

    import dataclasses as _dc
    sub = {}
    if not args.no_variants and world == 1:
        other = binding.RANK_POSITION if rank_mode == binding.RANK_SCORE else binding.RANK_SCORE
        p_other = _dc.replace(params, rank_mode=other)
        sub["score_mode" if other == binding.RANK_SCORE else "position_mode"] = variant_record(p_other, [d["q"] for d in layers])
        if cfg.window > 1:
            p_w1 = _dc.replace(params, window=1)
            sub["window_1"] = variant_record(p_w1, [d["q"][:, :, -1:, :].contiguous() for d in layers])
        step()                                   # leave the headline setting's budgets behind for what follows
        torch.cuda.synchronize()

    # what traffic of this shape can reach on the device: a read-only stream over one layer's K, and a row copy that
    # reads (1 + rho) and writes 2 rho of a layer's bytes, each swept over the layers like a stage
    def sweep_ms(call):
        for d in layers:
            call(d)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for d in layers:
                call(d)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (reps * L)

    rows_all = cfg.num_kv_heads * total
    kept_all = int(round(rho * rows_all))
    ceiling = {"rho": round(rho, 4),
               "how": "hand-written probes of the library: refree_sol_read_stream over a layer's K; refree_sol_row_mix "
                      "reads (1 + rho) and writes 2 rho of a layer's K/V bytes in 256-byte rows; swept over the layers; "
                      "each with vector loads/stores in registers and with the bulk-copy engine"}
    for tag, bulk in (("ldst", False), ("bulk", True)):
        read_ms = sweep_ms(lambda d: binding.refree_sol_read_stream(d["k"], bulk=bulk))
        mix_ms = sweep_ms(lambda d: binding.refree_sol_row_mix(d["k"], d["v"], d["k_out"], d["v_out"], rows_all, kept_all,
                                                               row, bulk=bulk))
        ceiling[f"read_stream_{tag}_gbs"] = round(rows_all * row / (read_ms * 1e-3) / 1e9, 1)
        ceiling[f"row_mix_{tag}_gbs"] = round((rows_all + 3 * kept_all) * row / (mix_ms * 1e-3) / 1e9, 1)
    ceiling["row_mix_gbs"] = max(ceiling["row_mix_ldst_gbs"], ceiling["row_mix_bulk_gbs"])
    step()                                       # the probes overwrote the outputs: put the pass's results back
    torch.cuda.synchronize()

    e2e = measure_e2e(binding, workloads, cfg, params, dev, L, total, cap, units, args)
    cpu_baseline = measure_cpu_baseline(cfg, rank_mode, total, args) if world == 1 and not args.no_cpu_baseline else None

    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 5), "blocks_timed": len(block_ms),
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
        "config": {"workload": cfg.name, "layers": L, "q_heads": cfg.num_q_heads, "kv_heads": cfg.num_kv_heads,
                   "head_dim": cfg.head_dim, "seq_lens": seq_lens if len(seq_lens) <= 8 else len(seq_lens),
                   "window": cfg.window, "sink": cfg.sink, "threshold": args.threshold, "rank_mode": args.rank_mode,
                   "scope": "head", "layout": "head_major",
                   "l2": f"each step sweeps {L} layers of distinct K/V buffers "
                         f"({L * 2 * cfg.num_kv_heads * total * row / 2**30:.1f} GiB), larger than L2",
                   "replicas": world},
        "gpu_launches": int(launches), "clocks": clocks, "e2e": e2e,
        "roofline": roofline, "roofline_pass": roofline_pass, "ceiling_gbs": ceiling["row_mix_gbs"], "ceiling": ceiling,
        **sub, "decode_attention": decode_line,
        "compact_inplace": inplace_line,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist_barrier(world)


def measure_e2e(binding, workloads, cfg, params, dev, L, total, cap, units, args):
    """Same metric through the host-buffer entry points: pinned host inputs are copied in, the pass
    runs, kept rows and budgets are copied back, every layer.  The headline is the pipelined call over
    a run of layers (copies in both directions overlap the pass); the one-layer-per-call figure is
    reported beside it."""
    n_lay = min(L, 16)
    row = cfg.head_dim * cfg.elem_bytes
    host = []
    for l in range(n_lay):
        lay = workloads.make_layer(cfg, l)
        host.append(dict(q=lay.q_win.pin_memory(), k=lay.k.pin_memory(), v=lay.v.pin_memory(),
                         ss=lay.seq_start, sl=lay.seq_len,
                         k_out=torch.empty(cap, cfg.head_dim, dtype=cfg.torch_dtype).pin_memory(),
                         v_out=torch.empty(cap, cfg.head_dim, dtype=cfg.torch_dtype).pin_memory(),
                         lengths=torch.zeros(units, dtype=torch.int32).pin_memory(),
                         offsets=torch.zeros(units + 1, dtype=torch.int64).pin_memory()))
    kv_elems = host[0]["k"].numel()
    reps = max(1, min(args.steps, 3))

    # one layer per call: copy in, pass, copy out, in sequence
    arena = torch.empty(binding.refree_host_arena_size(params, total, kv_elems, cap), dtype=torch.uint8, device=dev)

    def one(h):
        binding.refree_compress_layer_host(params, h["q"], h["k"], h["v"], h["ss"], h["sl"], total, h["k_out"],
                                           h["v_out"], cap, h["lengths"], h["offsets"], None, None, arena)

    for h in host[:2]:
        one(h)
    t0 = time.perf_counter()
    for h in host[:4]:
        one(h)
    per_layer_seq = (time.perf_counter() - t0) / min(4, n_lay)
    del arena

    # a run of layers per call, pipelined
    arena = torch.empty(binding.refree_host_pipeline_arena_size(params, total, kv_elems, cap), dtype=torch.uint8,
                        device=dev)
    cols = {key: [h[key] for h in host] for key in ("q", "k", "v", "k_out", "v_out", "lengths", "offsets")}

    def run():
        binding.refree_compress_layers_host(params, cols["q"], cols["k"], cols["v"], host[0]["ss"], host[0]["sl"], total,
                                            cols["k_out"], cols["v_out"], cap, cols["lengths"], cols["offsets"], arena)

    run()
    t0 = time.perf_counter()
    for _ in range(reps):
        run()
    per_layer = (time.perf_counter() - t0) / (reps * n_lay)
    d2h_layer = sum(int(h["offsets"][-1]) * 2 * row + units * 4 + (units + 1) * 8 + 4 for h in host) / n_lay
    h2d_layer = host[0]["q"].numel() * cfg.elem_bytes + 2 * kv_elems * cfg.elem_bytes + 8 * host[0]["sl"].numel() / n_lay
    return {"value": round(total / per_layer, 1), "unit": UNIT,
            "h2d_bytes_per_step": int(h2d_layer * L), "d2h_bytes_per_step": int(d2h_layer * L),
            "ms_per_step": round(per_layer * L * 1e3, 3),
            "one_layer_per_call": {"value": round(total / per_layer_seq, 1), "ms_per_step": round(per_layer_seq * L * 1e3, 3)},
            "how": f"refree_compress_layers_host (three-stream pipeline) on pinned host buffers, {n_lay} layers x "
                   f"{reps} calls, wall clock (the call returns when every layer is back in host memory), "
                   f"scaled to {L} layers; one_layer_per_call = refree_compress_layer_host, 4 layers"}


# --------------------------------------------------------- CPU oracle arm ----
def oracle_sample(cfg, rank_mode, layer_idx, heads, threshold=0.01):
    """Inputs of the oracle for `heads` KV heads of one layer of the workload."""
    from oracle import refree_oracle as orc
    from paper_2502_16886_b200 import workloads
    lay = workloads.make_layer(cfg, layer_idx)
    G = cfg.group
    total = lay.total_tokens
    p = orc.OracleParams(int(lay.seq_len.numel()), heads * G, heads, cfg.head_dim, window=cfg.window, sink=cfg.sink,
                         threshold=threshold, rank_mode=rank_mode, dtype=0 if cfg.dtype == "fp32" else 1,
                         k_strides=(0, cfg.head_dim, total * cfg.head_dim),
                         v_strides=(0, cfg.head_dim, total * cfg.head_dim))
    return p, lay.q_win[:, :heads * G].contiguous(), lay.k[:heads].contiguous(), lay.v[:heads].contiguous(), \
        lay.seq_start, lay.seq_len


def oracle_heads_for_budget(cfg, total, seconds=2.5):
    """KV heads per sample so that one oracle call takes about `seconds` on this host."""
    from oracle import refree_oracle as orc
    macs_per_head = cfg.group * cfg.window * total * cfg.head_dim
    rate = 1.2e9 * orc.num_threads()              # fp64 scalar multiply-adds per second, rough
    return max(1, min(cfg.num_kv_heads, int(seconds * rate / macs_per_head)))


def measure_cpu_baseline(cfg, rank_mode, total, args):
    from oracle import build as obuild, refree_oracle as orc
    obuild.build()
    heads = oracle_heads_for_budget(cfg, total)
    t_used, n_calls, layer = 0.0, 0, 0
    while t_used < 10.0 and n_calls < 8:
        inp = oracle_sample(cfg, rank_mode, layer % cfg.num_layers, heads, args.threshold)
        t0 = time.perf_counter()
        orc.compress_layer(*inp)
        t_used += time.perf_counter() - t0
        n_calls += 1
        layer += 1
    per_layer = t_used / n_calls * cfg.num_kv_heads / heads
    out = {"value": round(total / per_layer, 1), "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
           "sample": f"{n_calls} layer(s) of {cfg.name}, {heads} of {cfg.num_kv_heads} KV heads each, "
                     f"scaled to a full layer; {t_used:.1f}s of CPU time"}
    # one thread, on the 8K-token Llama3-8B-shaped cache: one KV head of one layer, scaled to the layer
    from paper_2502_16886_b200 import workloads
    cfg8 = workloads.get_config("llama3_8b_8k")
    threads = orc.num_threads()
    try:
        orc.set_num_threads(1)
        inp = oracle_sample(cfg8, rank_mode, 0, 1)
        t0 = time.perf_counter()
        orc.compress_layer(*inp)
        dt = time.perf_counter() - t0
    finally:
        orc.set_num_threads(threads)
    tot8 = sum(workloads.sequence_lengths(cfg8))
    out["single_thread_llama3_8b_8k"] = {"value": round(tot8 / (dt * cfg8.num_kv_heads), 1), "unit": UNIT, "cores": 1,
                                         "sample": f"1 of {cfg8.num_kv_heads} KV heads of one layer, scaled; {dt:.1f}s"}
    return out


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from oracle import build as obuild, refree_oracle as orc
    from paper_2502_16886_b200 import workloads
    obuild.build()
    cfg = workloads.get_config(args.workload)
    rank_mode = 1 if args.rank_mode == "score" else 0
    seq_lens = workloads.sequence_lengths(cfg)
    total = sum(seq_lens)
    heads = oracle_heads_for_budget(cfg, total, seconds=2.0)
    samples = [oracle_sample(cfg, rank_mode, l, heads, args.threshold) for l in range(min(2, cfg.num_layers))]
    for i in range(args.warmup):
        orc.compress_layer(*samples[i % len(samples)])
    t0 = time.perf_counter()
    for i in range(args.steps):
        orc.compress_layer(*samples[i % len(samples)])
    dt = (time.perf_counter() - t0) / args.steps
    per_layer = dt * cfg.num_kv_heads / heads
    value = round(total / per_layer, 1)
    sample = (f"one step = {heads} of {cfg.num_kv_heads} KV heads of one layer of {cfg.name} (a bounded sample of the "
              f"workload); value = tokens / (step time x {cfg.num_kv_heads}/{heads}); host-resident inputs")
    row = cfg.head_dim * cfg.elem_bytes
    L = cfg.num_layers
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 3),
            "scaled_to_full_layer": {"ms_per_layer": round(per_layer * 1e3, 3), "kv_heads_timed": heads,
                                     "kv_heads": cfg.num_kv_heads},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "layers": L, "q_heads": cfg.num_q_heads, "kv_heads": cfg.num_kv_heads,
                       "head_dim": cfg.head_dim, "seq_lens": seq_lens if len(seq_lens) <= 8 else len(seq_lens),
                       "window": cfg.window, "sink": cfg.sink, "threshold": args.threshold, "rank_mode": args.rank_mode,
                       "scope": "head", "layout": "head_major",
                       "l2": f"each step sweeps {L} layers of distinct K/V buffers "
                             f"({L * 2 * cfg.num_kv_heads * total * row / 2**30:.1f} GiB), larger than L2",
                       "replicas": world},
            "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """The paper's ablations as a second workload (Section 4.4: the window k as a share of n; Section 3.2: T between
    0.1 % and 10 %): one refree_compress_layers call over a cut of the 8K cache per point.  A window whose row count
    the library does not take is reported as unsupported, not skipped."""
    from paper_2502_16886_b200 import binding, build, workloads
    import dataclasses
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    dev = torch.device("cuda", 0)
    build.build()
    binding.lib()
    base = workloads.get_config("llama3_8b_8k")
    L = args.layers or 8
    n = workloads.sequence_lengths(base)[0]
    points = []
    for window in (1, max(1, round(0.01 * n)), round(0.05 * n), round(0.10 * n)):
        cfg = dataclasses.replace(base, window=window)
        rows = cfg.group * window
        if rows > 32768:
            points += [{"window": window, "threshold": t, "status": "unsupported: G * window = %d rows > 32768" % rows}
                       for t in (0.001, 0.01, 0.1)]
            continue
        lays = [workloads.make_layer(cfg, l) for l in range(L)]
        total = lays[0].total_tokens
        cap = cfg.num_kv_heads * total
        units = cfg.num_kv_heads
        dv = [dict(q=x.q_win.to(dev), k=x.k.to(dev), v=x.v.to(dev),
                   k_out=torch.empty(cap, cfg.head_dim, dtype=cfg.torch_dtype, device=dev),
                   v_out=torch.empty(cap, cfg.head_dim, dtype=cfg.torch_dtype, device=dev),
                   lengths=torch.zeros(units, dtype=torch.int32, device=dev),
                   offsets=torch.zeros(units + 1, dtype=torch.int64, device=dev)) for x in lays]
        ss, sl = lays[0].seq_start.to(dev), lays[0].seq_len.to(dev)
        ptrs = binding.LayerPointers(*[[d[key] for d in dv] for key in ("q", "k", "v", "k_out", "v_out", "lengths", "offsets")])
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        for t in (0.001, 0.01, 0.1):
            p = binding.params_for(cfg, lays[0], threshold=t)
            ws = torch.empty(binding.refree_layers_workspace_size(p, total), dtype=torch.uint8, device=dev)

            def run():
                binding.refree_compress_layers(p, ptrs, ss, sl, total, cap, ws, status)
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                run()
            e1.record()
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            ms = e0.elapsed_time(e1) / (10 * L)
            rho = sum(int(d["lengths"].sum()) for d in dv) / (L * cap)
            points.append({"window": window, "threshold": t, "us_per_layer": round(ms * 1e3, 2),
                           "tokens_per_s_per_layer": round(total / (ms * 1e-3), 1), "kept_ratio": round(rho, 4)})
        del dv, lays
        torch.cuda.empty_cache()
    print(json.dumps({"metric": METRIC, "unit": UNIT, "sweep": "threshold x window on llama3_8b_8k (Section 4.4, Section 3.2)",
                      "layers": L, "rank_mode": "position", "data": "synthetic", "points": points}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--rank-mode", choices=["position", "score"], default="position")
    ap.add_argument("--layers", type=int, default=0, help="debugging: use fewer layers than the config")
    ap.add_argument("--window", type=int, default=0, help="override the config's observation window (paper default: 1)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the score-ranking and single-row sub-records")
    ap.add_argument("--threshold", type=float, default=0.01, help="the stopping rule's T (paper: 1 %%)")
    ap.add_argument("--sweep", action="store_true",
                    help="second workload: T in {0.1 %%, 1 %%, 10 %%} x window in {1, 1 %%n, 5 %%n, 10 %%n} on the 8K cache")
    ap.add_argument("--per-layer-calls", action="store_true",
                    help="time one refree_compress_layer call per layer instead of one refree_compress_layers call per step")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args)
    else:
        args.steps = args.steps if args.steps is not None else 200
        args.warmup = args.warmup if args.warmup is not None else 5
        run_ours(args)


if __name__ == "__main__":
    main()
