#!/usr/bin/env python
"""Benchmark of the sequence-split decode-attention path (one JSON line on stdout, printed by rank 0).

A "step" is one decode step of the whole path over one batch: for every layer, append one new K/V token
per sequence (write-time routing into the D-window), attend the GPU-side share (split-K attention kernel +
LSE reduce), and merge with the CPU-side partial (LSE merge kernel).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Metric: KV-tokens/s of GPU-share decode attention, where one KV-token is one token of one layer's cache
(all KV heads) attended by all query heads; bytes = KV-tokens x bytes per token per layer.
With N > 1 every rank runs an independent replica on its own GPU (the path has no exchange step);
`value` is the sum over ranks divided by the slowest rank's time.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2609_14507_b200 import synth  # noqa: E402

METRIC = "gpu_share_decode_attn_kv_tokens_per_s"
UNIT = "KV-tokens/s"

WORKLOADS = {
    # BASELINE config 2: Mixtral-8x7B-shaped attention, 32 layers, batch 16, 32K context, CPU share 25 %
    "mixtral-8x7b-bs16-32k-cpu25": dict(shape=synth.MIXTRAL, batch=16, ctx=32768, share=(1, 4), cfg_id=2),
    # BASELINE config 3 at CPU share 0: Qwen3-30B-A3B-shaped attention, 48 layers, batch 16, 32K context
    "qwen3-30b-a3b-bs16-32k-cpu0": dict(shape=synth.QWEN3, batch=16, ctx=32768, share=(0, 1), cfg_id=3),
    "qwen3-30b-a3b-bs16-32k-cpu10": dict(shape=synth.QWEN3, batch=16, ctx=32768, share=(1, 10), cfg_id=3),
    "qwen3-30b-a3b-bs16-32k-cpu30": dict(shape=synth.QWEN3, batch=16, ctx=32768, share=(3, 10), cfg_id=3),
    "qwen3-30b-a3b-bs16-32k-cpu50": dict(shape=synth.QWEN3, batch=16, ctx=32768, share=(1, 2), cfg_id=3),
    "qwen3-30b-a3b-bs16-32k-cpu70": dict(shape=synth.QWEN3, batch=16, ctx=32768, share=(7, 10), cfg_id=3),
    # two layers of config 2: a few GB on the device, still far larger than L2 -- the size used for ncu captures
    "mixtral-2layers-bs16-32k-cpu25": dict(shape=synth.Shape("mixtral-2l", "gqa", 2, 32, 8, 128, 128, 128 ** -0.5), batch=16,
                                           ctx=32768, share=(1, 4), cfg_id=2),
    "qwen3-2layers-bs16-32k-cpu0": dict(shape=synth.Shape("qwen3-2l", "gqa", 2, 32, 4, 128, 128, 128 ** -0.5), batch=16,
                                        ctx=32768, share=(0, 1), cfg_id=3),
    # BASELINE config 4: DeepSeek-V2-Lite-shaped MLA decode, 27 layers, batch 8, 128K context, CPU share 40 %
    "deepseek-v2-lite-mla-bs8-128k-cpu40": dict(shape=synth.DSV2_LITE, batch=8, ctx=131072, share=(2, 5), cfg_id=4),
    "deepseek-v2-lite-mla-2layers-bs8-128k-cpu40": dict(shape=synth.Shape("dsv2-2l", "mla", 2, 16, 1, 576, 512, 192 ** -0.5),
                                                        batch=8, ctx=131072, share=(2, 5), cfg_id=4),
    # BASELINE config 1 (single layer, batch 1, 4K): latency-bound, for quick checks
    "small-gqa-bs1-4k-cpu50": dict(shape=synth.SMALL_GQA, batch=1, ctx=4096, share=(1, 2), cfg_id=1),
}
# dram__bytes_read.sum + dram__bytes_write.sum of one attention-kernel launch, read from one ncu capture per kernel
# (taken on the 2-layer case of each shape, whose per-layer launch is the full-size workload's launch): read + write bytes.
DRAM_TRAFFIC_PER_LAUNCH = {
    "mixtral-8x7b-bs16-32k-cpu25": 1615.2e6 + 4.5e6,
    "mixtral-2layers-bs16-32k-cpu25": 1615.2e6 + 4.5e6,
    "qwen3-30b-a3b-bs16-32k-cpu0": 1076.1e6 + 3.9e6,
    "qwen3-2layers-bs16-32k-cpu0": 1076.1e6 + 3.9e6,
    "deepseek-v2-lite-mla-bs8-128k-cpu40": 725.7e6 + 4.1e6,
    "deepseek-v2-lite-mla-2layers-bs8-128k-cpu40": 725.7e6 + 4.1e6,
}
DEFAULT_WORKLOAD = "mixtral-8x7b-bs16-32k-cpu25"
# Short runs of the other BASELINE configurations, reported beside the default line (rank 0, one GPU): config 3 at CPU
# share 0 and 70 %, config 4 (compressed-latent kernel), config 5 at CPU share 0.
OTHER_CONFIGS = ["qwen3-30b-a3b-bs16-32k-cpu0", "qwen3-30b-a3b-bs16-32k-cpu70", "deepseek-v2-lite-mla-bs8-128k-cpu40",
                 "qwen3-ragged-bs64-1m-cpu0"]
BLOCK, WINDOW = 64, 256

# BASELINE config 5: Qwen3 shape, 48 layers, batch 64, ragged context lengths uniform in [8192, 24576] (about 1M tokens
# in all), CPU share swept 0 .. 90 %.  Every sequence's part of the resident ring is sized for that sequence
# (ipkv_config.resident_tokens_by_seq), so the batch holds its 103 GB at share 0 and not the longest sequence's ring 64 times.
for _pct in range(0, 100, 10):
    WORKLOADS[f"qwen3-ragged-bs64-1m-cpu{_pct}"] = dict(
        shape=synth.QWEN3, batch=64, ctx=24576, share=(_pct, 100), cfg_id=5, lens=synth.ragged_lengths(5, 64, 8192, 24576))
WORKLOADS["qwen3-ragged-bs64-1m-2layers-cpu30"] = dict(
    shape=synth.Shape("qwen3-2l", "gqa", 2, 32, 4, 128, 128, 128 ** -0.5), batch=64, ctx=24576, share=(3, 10), cfg_id=5,
    lens=synth.ragged_lengths(5, 64, 8192, 24576))


# Load reading of config 3 ("host-share chunks streamed H2D from pinned memory"): the oldest `stream_pct` % of every
# sequence's P share is NOT device-resident; it lives in pinned host memory and is streamed through the PP slots on a
# side stream each step while the resident rest is attended. 2 layers: the pinned host copy of P is 1 GB per layer.
for _pct in (10, 30, 50, 70, 100):
    WORKLOADS[f"qwen3-2layers-bs16-32k-stream{_pct}"] = dict(
        shape=synth.Shape("qwen3-2l", "gqa", 2, 32, 4, 128, 128, 128 ** -0.5), batch=16, ctx=32768, share=(0, 1), cfg_id=3,
        stream_pct=_pct, chunk_tokens=4096)


# Decode with the host copies of U and P switched ON (pinned P, unpinned U): every 256 steps each layer evicts its
# D-window (8.4 MB per layer, device -> host). Used with --latency to look at per-step latency across evictions
# (the paper reports P99/P50 = 1.03 over 1000 steps for this shape at batch 8, 8K context).
for _pct, _share in ((0, (0, 1)), (50, (1, 2)), (100, (1, 1))):
    WORKLOADS[f"qwen3-30b-a3b-bs8-8k-cpu{_pct}-hostcopies"] = dict(shape=synth.QWEN3, batch=8, ctx=8192, share=_share, cfg_id=3,
                                                                   host_copies=True)
# The same decode with other eviction windows D (the paper: any D in 256-1024 leaves the steady state unchanged,
# Sec. 4.2) and with P grown batch by batch, each batch's memory pinned one window ahead by a helper thread
# (Sec. 4.3, Sec. 7.7), instead of pinned in full at start-up.  Used with --latency.
for _d in (256, 512, 1024):
    for _pct, _share in ((0, (0, 1)), (50, (1, 2))):
        WORKLOADS[f"qwen3-30b-a3b-bs8-8k-cpu{_pct}-hostcopies-d{_d}"] = dict(
            shape=synth.QWEN3, batch=8, ctx=8192, share=_share, cfg_id=3, host_copies=True, window=_d, chunk_tokens=1024)
        WORKLOADS[f"qwen3-30b-a3b-bs8-8k-cpu{_pct}-growp-d{_d}"] = dict(
            shape=synth.QWEN3, batch=8, ctx=8192, share=_share, cfg_id=3, host_copies=True, window=_d, chunk_tokens=1024, grow_p=True)


def seq_lens(wl):
    """Context length of every sequence of the batch."""
    return [int(x) for x in wl["lens"]] if "lens" in wl else [wl["ctx"]] * wl["batch"]


def cpu_tokens(n, num0, den0):
    """Prefill tokens the CPU side takes: whole blocks, floored (the library's and the oracle's rule)."""
    return BLOCK * ((n // BLOCK) * num0 // den0)


def kv_seed(wl, layer, seq, rank=0):
    return 1000 * wl["cfg_id"] + layer * wl["batch"] + seq + 100000 * rank


def make_cache(wl, device_index, decode_steps):
    """The cache of a workload as the benchmark times it: GPU-side share HBM-resident, host copies of U and P off."""
    from paper_2609_14507_b200 import binding
    sh = wl["shape"]
    num0, den0 = wl["share"]
    longest = max(seq_lens(wl))
    window = wl.get("window", WINDOW)
    grow = window * (decode_steps // window + 2)
    p_cap = longest - cpu_tokens(longest, num0, den0) + grow if num0 < den0 else grow
    p_cap = max(p_cap, max(n - cpu_tokens(n, num0, den0) for n in seq_lens(wl)) + grow)
    kind = binding.MLA if sh.kind == "mla" else binding.GQA
    resident, flags = p_cap, binding.FLAG_NO_HOST_U | binding.FLAG_NO_HOST_P
    by_seq = None
    if "lens" in wl and not wl.get("host_copies") and "stream_pct" not in wl:
        # ragged batch: every sequence's ring holds its own GPU-side share plus the decode steps' growth
        by_seq = [n - cpu_tokens(n, num0, den0) + grow if num0 < den0 else grow for n in seq_lens(wl)]
    if wl.get("host_copies"):
        flags = 0
    if "stream_pct" in wl:
        # keep the newest (100 - stream_pct) % of the prefill's P share resident; P itself lives in pinned host memory
        resident = BLOCK * (((longest - cpu_tokens(longest, num0, den0)) * (100 - wl["stream_pct"]) // 100) // BLOCK)
        flags = binding.FLAG_NO_HOST_U
    p_initial = 0
    if wl.get("grow_p"):
        # create pins the prefill's share (rounded up to whole chunks); decode batches get their memory as they come
        chunk = wl.get("chunk_tokens", 512)
        p_initial = -(-(longest - cpu_tokens(longest, num0, den0)) // chunk) * chunk
        p_cap = max(p_cap, p_initial)
        flags |= binding.FLAG_GROW_P
    cfg = binding.make_config(kind, sh.n_layers, wl["batch"], sh.n_q_heads, sh.n_kv_heads, sh.dim_qk, sh.dim_v,
                              block_tokens=BLOCK, window_tokens=window, chunk_tokens=wl.get("chunk_tokens", 512), n_slots=2,
                              p_initial_tokens_per_seq=p_initial,
                              max_u_tokens_per_seq=longest + grow, max_p_tokens_per_seq=p_cap, resident_tokens_per_seq=resident,
                              resident_tokens_by_seq=by_seq,
                              softmax_scale=sh.scale, share_num=num0, share_den=den0, device=device_index, flags=flags)
    return binding.Cache(cfg)


def populate(cache, wl, dev, rank=0):
    """Prefill every (layer, sequence) with seeded N(0,1) K/V, routed in one shot at the workload's share."""
    import torch
    sh = wl["shape"]
    num0, den0 = wl["share"]
    for layer in range(sh.n_layers):
        for s, n in enumerate(seq_lens(wl)):
            k, v = synth.device_kv(sh, n, kv_seed(wl, layer, s, rank), dev)
            cache.append_bulk(layer, s, k, v, n, num0, den0)
        torch.cuda.synchronize()


def reduce_over_ranks(x, op, device):
    """All-reduce of one float over the ranks of the default process group ("max" or "sum"); identity for one rank.
    Replicas do not exchange data: this only combines the timings (max) and the work counts (sum) of the ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([float(x)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX if op == "max" else dist.ReduceOp.SUM)
    return float(t.item())


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index, self.rows, self.proc, self.thread, self.t_mark = gpu_index, [], None, None, 0.0

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def mark(self):
        """Start of the load (the first warm-up step): earlier samples are dropped."""
        self.t_mark = time.time()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        if self.thread:
            self.thread.join(timeout=2)
        sm, mx, watts, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, r in self.rows:
            if len(r) < 7 or ts < self.t_mark:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            try:
                watts.append(float(r[2]))
            except ValueError:
                pass
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w": statistics.median(watts) if watts else None}


def oracle_sample(wl, seconds_target=15.0, threads=None):
    """Time the float64 oracle, as it stands, on a bounded sample of the workload: the GPU-side share of whole
    (layer, sequence) pairs (all KV heads, all query heads), as many pairs as fit the time target."""
    import torch
    from oracle import c_oracle
    sh = wl["shape"]
    num0, den0 = wl["share"]
    lens = seq_lens(wl)
    if threads:
        c_oracle.set_threads(threads)
    dev = "cuda:0" if torch.cuda.is_available() else None
    done_tokens, t_total, n_pairs = 0, 0.0, 0
    while True:
        layer, s = divmod(n_pairs, wl["batch"])
        n = lens[s]
        seed = kv_seed(wl, layer, s)
        if dev:
            kd, vd = synth.device_kv(sh, n, seed, dev)
            k, v = synth.torch_bits(kd), (synth.torch_bits(vd) if vd is not None else None)
            q = synth.torch_bits(synth.device_q(sh, 1, seed + 500000, dev))[0]
        else:
            k, v = synth.host_kv(sh, n, seed)
            q = synth.host_q(sh, 1, seed + 500000)[0]
        idx = np.arange(cpu_tokens(n, num0, den0), n)
        t0 = time.perf_counter()
        c_oracle.attend(q, k, sh.dim_v if v is None else v, idx, float(np.float32(sh.scale)))
        dt = time.perf_counter() - t0
        done_tokens += idx.size
        t_total += dt
        n_pairs += 1
        if t_total >= seconds_target or n_pairs >= sh.n_layers * wl["batch"]:
            break
    # the same code on one thread, on the last pair of the sample
    used = c_oracle.num_threads()
    c_oracle.set_threads(1)
    t0 = time.perf_counter()
    c_oracle.attend(q, k, sh.dim_v if v is None else v, idx, float(np.float32(sh.scale)))
    single = idx.size / (time.perf_counter() - t0)
    c_oracle.set_threads(used)
    return dict(value=done_tokens / t_total, unit=UNIT, cores=used, kind="oracle", host_cpus=os.cpu_count(), single_thread_value=single,
                sample=f"{n_pairs} of {sh.n_layers * wl['batch']} (layer, sequence) pairs, GPU-side share ({done_tokens} KV-tokens "
                       f"in all), all heads; {t_total:.1f} s of float64 C++ (OpenMP over query heads)")


def other_config(name, steps=10, warmup=3):
    """One short run of another workload in a process of its own (its cache needs the whole device); the headline
    figures of its JSON line."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--workload", name, "--steps", str(steps), "--warmup", str(warmup),
           "--no-cpu-baseline", "--no-read-ceiling", "--no-other-configs"]
    try:
        r = subprocess.run(cmd, capture_output=True, text=True, timeout=900, cwd=ROOT)
        d = json.loads(r.stdout.strip().splitlines()[-1])
    except Exception as e:                                  # noqa: BLE001 - reported in the line, the headline stands
        return {"workload": name, "error": repr(e)[:200]}
    rf = d["roofline"]
    return {"workload": name, "steps": steps, "ms_per_step": d["ms_per_step"], "value": d["value"], "kernel": rf["kernel"],
            "achieved": rf["achieved"], "frac": rf["frac"], "avg_launch_us": rf["avg_launch_us"], "step_gbs": d["step_gbs"],
            "e2e_ms_per_step": d["e2e"]["ms_per_step"] if d.get("e2e") else None,
            "sm_mhz": (d.get("clocks") or {}).get("sm_mhz"), "layers": d["config"]["layers"]}


def replica_envs(n, port, base_env=None):
    """Environment of each of n replica processes on this node (one per GPU): what a launcher would have set."""
    base = dict(os.environ if base_env is None else base_env)
    return [dict(base, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
            for r in range(n)]


def spawn_replicas(n, argv):
    """`bench.py --gpus N` without a launcher: start the N replica processes here (rank 0 prints the JSON line) and wait."""
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    procs = [subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py")] + argv, env=env, cwd=ROOT)
             for env in replica_envs(n, port)]
    codes = [p.wait() for p in procs]
    return max(codes, key=abs) if any(codes) else 0


def workload_config(name, wl):
    """What the workload is, from its table entry alone: both arms print the same object for the same workload.
    What a particular run chose (schedule, splits, timing cadence) goes under the line's "run" key instead."""
    sh, B = wl["shape"], wl["batch"]
    num0, den0 = wl["share"]
    lens = seq_lens(wl)
    n_cpu = sum(cpu_tokens(n, num0, den0) for n in lens) // B
    n_gpu0 = sum(lens) // B - n_cpu
    bpt = sh.bytes_per_token
    # every layer reads its own KV, so one step sweeps all layers' bytes before a byte is read again
    layer_bytes = sum(n - cpu_tokens(n, num0, den0) + 1 for n in lens) * bpt
    step_bytes = layer_bytes * sh.n_layers
    if step_bytes > 2 * (126 << 20):
        l2_note = "inputs larger than L2 (each layer reads its own %.2f GB; %.2f GB per step)" % (layer_bytes / 1e9, step_bytes / 1e9)
    else:
        l2_note = "NOT flushed: the %.1f MB a step reads stay L2-resident between steps; a latency case, not a bandwidth number" % (step_bytes / 1e6)
    gpu_share, copies = "HBM-resident", "off (benchmark)"
    if wl.get("host_copies"):
        copies = "on (P pinned, U unpinned); write-back on a copy stream"
    if wl.get("grow_p"):
        copies += "; P grown batch by batch, pinned one window ahead by a helper thread"
    if "stream_pct" in wl:
        gpu_share = "%d %% streamed H2D from pinned host memory each step, rest HBM-resident" % wl["stream_pct"]
        copies = "P on (pinned), U off"
    return {"workload": name, "layers": sh.n_layers, "batch": B,
            "context": wl["ctx"] if "lens" not in wl else f"ragged {min(lens)}..{max(lens)} (sum {sum(lens)})",
            "cpu_share": f"{num0}/{den0}", "gpu_share_tokens_per_seq_mean": n_gpu0 + 1, "bytes_per_kv_token": bpt,
            "block_tokens": BLOCK, "window_tokens": wl.get("window", WINDOW), "gpu_share": gpu_share,
            "host_copies_of_U_and_P": copies, "cpu_partial": "synthetic values", "l2": l2_note, "multi_gpu": "replicas only"}


def run_reference(args, wl, name):
    """--impl reference: the oracle on the host cores, on the same workload and metric; each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = []
    for _ in range(args.warmup):
        oracle_sample(wl, seconds_target=1.0)
    info = None
    for _ in range(args.steps):
        info = oracle_sample(wl, seconds_target=max(2.0, min(15.0, 120.0 / max(1, args.steps))))
        per_step.append(info["value"])
    value = float(np.mean(per_step))
    info["value"] = value
    sh = wl["shape"]
    n_tok = sh.n_layers * sum(n - cpu_tokens(n, *wl["share"]) + 1 for n in seq_lens(wl))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * n_tok / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(name, wl),
        "cpu_baseline": info, "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def h2d_microbench():
    """Context numbers for the load path (the paper's Sec. 3.1-3.2 and Sec. 5.3 footnote, re-measured on this machine):
    host-to-device bandwidth by transfer size, pinned against pageable memory, and one contiguous copy against the
    same bytes as strided rows (cudaMemcpy2D, 4 KB rows at an 8 KB pitch, the shape of a per-head slice of a
    token-major cache)."""
    import torch
    dev = "cuda:0"
    torch.cuda.set_device(0)

    def timed(fn, reps=5):
        best = 1e9
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(); fn(); b.record(); torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        return best * 1e-3

    out = {"pinned_gbs": {}, "pageable_gbs": {}}
    dst = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    for label, size in (("192KB", 192 << 10), ("1MB", 1 << 20), ("8MB", 8 << 20), ("64MB", 64 << 20), ("256MB", 256 << 20)):
        hp = torch.empty(size, dtype=torch.uint8).pin_memory()
        hu = torch.empty(size, dtype=torch.uint8)
        hu.fill_(1)
        out["pinned_gbs"][label] = size / timed(lambda: dst[:size].copy_(hp, non_blocking=True)) / 1e9
        out["pageable_gbs"][label] = size / timed(lambda: dst[:size].copy_(hu, non_blocking=True)) / 1e9
    # contiguous against strided: 64 MB as 16384 rows of 4 KB, source pitch 8 KB
    rows, width = 16384, 4096
    src = torch.empty((rows, 2 * width), dtype=torch.uint8).pin_memory()
    d2 = torch.empty((rows, width), dtype=torch.uint8, device=dev)
    out["contiguous_64MB_gbs"] = rows * width / timed(lambda: d2.copy_(src.view(-1)[:rows * width].view(rows, width), non_blocking=True)) / 1e9
    out["strided_64MB_gbs"] = rows * width / timed(lambda: d2.copy_(src[:, :width], non_blocking=True)) / 1e9
    print(json.dumps({"h2d_microbench": out, "note": "context for the streamed mode; paper (A100, PCIe Gen4): pinned 25.4 GB/s at 8 MB, "
                      "22.2 at 1 MB, 8.7 at 192 KB; pageable 10; strided 4.6"}))


def cpu_engine_microbench():
    """The CPU-side engine (in-place attention over the unpinned region, Sec. 6.1) on the host cores of this machine: the
    quantity the roofline policy calls A (seconds per CPU-side KV token, Eq. 1).  Qwen3 and DeepSeek-V2-Lite shapes,
    one layer; the CPU share sits in U (PLAIN blocks, unpinned), written there by the library's own prefill routing."""
    import torch
    from paper_2609_14507_b200 import binding
    dev = "cuda:0"
    torch.cuda.set_device(0)
    out = {}
    for name, sh, batch, n_u in (("qwen3 (GQA 32/4, d 128)", synth.QWEN3, 16, 16384), ("deepseek-v2-lite (latent 576/512, 16 heads)", synth.DSV2_LITE, 8, 16384)):
        kind = binding.MLA if sh.kind == "mla" else binding.GQA
        cfg = binding.make_config(kind, 1, batch, sh.n_q_heads, sh.n_kv_heads, sh.dim_qk, sh.dim_v, block_tokens=BLOCK, window_tokens=WINDOW,
                                  chunk_tokens=512, max_u_tokens_per_seq=n_u, max_p_tokens_per_seq=2 * WINDOW, resident_tokens_per_seq=2 * WINDOW,
                                  softmax_scale=sh.scale, flags=binding.FLAG_NO_HOST_P)
        with binding.Cache(cfg) as cache:
            for s_ in range(batch):
                k, v = synth.device_kv(sh, n_u + WINDOW, 4242 + s_, dev)
                cache.append_bulk(0, s_, k, v, n_u + WINDOW, n_u, n_u + WINDOW)      # the first n_u tokens go to U
            torch.cuda.synchronize()
            cache.get_stats()                                                          # drains the write-back stream
            q = torch.randn((batch, sh.n_q_heads, sh.dim_qk)).to(torch.bfloat16)
            o = torch.zeros((batch, sh.n_q_heads, sh.dim_v)); lse = torch.zeros((batch, sh.n_q_heads))
            ids = list(range(batch))
            times = []
            for _ in range(6):
                t0 = time.perf_counter()
                cache.attend_cpu(0, ids, q, o, lse)
                times.append(time.perf_counter() - t0)
            t = statistics.median(times[1:])
            tokens = batch * n_u
            out[name] = {"cpu_tokens": tokens, "seconds": t, "kv_tokens_per_s": tokens / t, "gb_per_s": tokens * sh.bytes_per_token / t / 1e9,
                         "A_seconds_per_token_per_sequence_batch": t / n_u, "threads": os.cpu_count()}
    print(json.dumps({"cpu_engine_microbench": out}))


def two_engine_bench(steps=None, resident=False):
    """The paper's whole decode step with both engines live (Sec. 4.2, Eq. 1-2): per layer a host thread runs the CPU
    engine over region U in place WHILE the GPU attends P and the D-window; one join per layer; the CPU engine's wall
    time feeds the policy's sliding window and once per D-window the policy's marginal share goes to ipkv_set_share.
    Qwen3 shape, batch 8, 8K context, 12 layers, host copies of U and P on.  By default the GPU side is the paper's:
    nothing of P stays on the device, every chunk is streamed from pinned host memory through two slots each step
    (`--two-engine-resident` keeps P in HBM instead: the B200 adaptation, where the GPU side is so much cheaper per
    token than the CPU side that Eq. 2 sends the share to zero)."""
    import queue
    import torch
    from paper_2609_14507_b200 import binding
    dev = "cuda:0"
    torch.cuda.set_device(0)
    sh = synth.Shape("qwen3-12l", "gqa", 12, 32, 4, 128, 128, 128 ** -0.5)
    NL, Bn, L0, D, den = sh.n_layers, 8, 8192, 64, 64
    steps = steps or 5 * D
    cap = L0 + steps + 2 * D
    num0 = den // 2                                          # prefill share 1/2; the decode batches follow the policy
    policy = None                                            # created after the first steps have calibrated B
    cfg = binding.make_config(binding.GQA, NL, Bn, sh.n_q_heads, sh.n_kv_heads, sh.dim_qk, sh.dim_v, block_tokens=BLOCK,
                              window_tokens=D, chunk_tokens=1024, n_slots=2, max_u_tokens_per_seq=cap, max_p_tokens_per_seq=cap,
                              resident_tokens_per_seq=cap if resident else 0, softmax_scale=sh.scale, share_num=num0, share_den=den,
                              flags=0)
    ids = list(range(Bn))
    with binding.Cache(cfg) as cache:
        for layer in range(NL):
            for s_ in range(Bn):
                k, v = synth.device_kv(sh, L0, 31000 + layer * Bn + s_, dev)
                cache.append_bulk(layer, s_, k, v, L0, num0, den)
            torch.cuda.synchronize()
        g = torch.Generator(device=dev); g.manual_seed(5)
        bf = torch.bfloat16
        q = torch.randn((NL, Bn, sh.n_q_heads, sh.dim_qk), generator=g, device=dev).to(bf)
        kn = torch.randn((NL, Bn, sh.n_kv_heads, sh.dim_qk), generator=g, device=dev).to(bf)
        vn = torch.randn((NL, Bn, sh.n_kv_heads, sh.dim_v), generator=g, device=dev).to(bf)
        q_host = q.cpu().pin_memory()
        rows, dv = Bn * sh.n_q_heads, sh.dim_v
        o_cpu = torch.zeros((NL, rows, dv)).pin_memory(); l_cpu = torch.zeros((NL, rows)).pin_memory()
        o_gpu = torch.zeros((rows, dv), device=dev); l_gpu = torch.zeros((rows,), device=dev)
        out = torch.zeros((NL, rows, dv), device=dev); out_lse = torch.zeros((rows,), device=dev)
        jobs, done = queue.Queue(), queue.Queue()

        def worker():                                       # the CPU engine's thread: one layer per job
            while True:
                layer = jobs.get()
                if layer is None:
                    return
                t0 = time.perf_counter()
                cache.attend_cpu(layer, ids, q_host[layer], o_cpu[layer].view(Bn, sh.n_q_heads, dv), l_cpu[layer].view(Bn, sh.n_q_heads))
                done.put(time.perf_counter() - t0)

        th = threading.Thread(target=worker, daemon=True)
        th.start()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(NL)]
        rec, shares = [], [num0]
        for step in range(steps):
            for layer in range(NL):                         # routing first: nothing may change it while the CPU engine reads it
                cache.append(layer, ids, kn[layer], vn[layer])
            torch.cuda.synchronize()
            t_cpu = 0.0
            w0 = time.perf_counter()
            for layer in range(NL):
                jobs.put(layer)
                ev[layer][0].record()
                cache.attend_gpu(layer, ids, q[layer], o_gpu.view(Bn, sh.n_q_heads, dv), l_gpu.view(Bn, sh.n_q_heads))
                ev[layer][1].record()
                t_cpu += done.get()                         # the join: both partials of the layer exist
                ev[layer][2].record()
                cache.merge(rows, dv, [o_gpu, o_cpu[layer]], [l_gpu, l_cpu[layer]], out[layer], out_lse)
                ev[layer][3].record()
            torch.cuda.synchronize()
            wall = time.perf_counter() - w0
            t_gpu = sum(ev[l][0].elapsed_time(ev[l][1]) for l in range(NL)) * 1e-3
            t_merge = sum(ev[l][2].elapsed_time(ev[l][3]) for l in range(NL)) * 1e-3
            c = [cache.counts(0, s_) for s_ in ids]
            n_u = sum(x["n_u"] for x in c); n_g = sum(x["n_p"] + x["n_w"] for x in c)
            if policy is None and step == 2:
                # B (seconds per GPU-side KV token of one layer) is calibrated once, from the step just timed; A starts equal
                b_cal = t_gpu / NL / max(1.0, n_g)
                policy = binding.Policy(A=b_cal, B=b_cal, C_cpu=0.0, C_gpu=0.0, window_steps=256, share_den=den)
            if policy is not None:
                policy.observe(t_cpu / NL, float(n_u))     # one layer's CPU latency and the CPU-side tokens it attended
            rec.append((wall, t_cpu, t_gpu, t_merge, n_u, n_g))
            if (step + 1) % D == 0:
                num, model = policy.update()
                cache.set_share(num)
                shares.append(num)
        jobs.put(None)
        th.join()
        st = cache.get_stats()
    tail = rec[len(rec) // 2:]                               # the second half: the policy has settled
    med = lambda i: statistics.median(r[i] for r in tail)
    wall, t_cpu, t_gpu, t_merge, n_u, n_g = (med(i) for i in range(6))
    # the GPU-side time seen by the events contains the wait for the CPU side's join only through the merge: t_gpu is the
    # attention call's own device time (for the streamed mode: copies and kernels of every chunk)
    A = t_cpu / NL / max(1.0, n_u); Bc = t_gpu / NL / max(1.0, n_g)
    L = (n_u + n_g) / Bn
    r_eq2 = binding.ipkv_roofline_share(A, Bc, 0.0, 0.0, L)
    print(json.dumps({"two_engine": {
        "workload": "qwen3 shape, %d layers, batch %d, context %d + %d decode steps, D %d, GPU side %s" % (
            NL, Bn, L0, steps, D, "HBM-resident" if resident else "streamed from pinned host memory (paper mode)"),
        "per_step_ms": {"wall": wall * 1e3, "sum_T_cpu": t_cpu * 1e3, "sum_T_gpu": t_gpu * 1e3, "sum_T_merge": t_merge * 1e3,
                        "eq1_max_plus_merge": (max(t_cpu, t_gpu) + t_merge) * 1e3},
        "wall_over_eq1": wall / (max(t_cpu, t_gpu) + t_merge),
        "cpu_share_now": n_u / max(1.0, n_u + n_g), "share_numerators_over_%d" % den: shares,
        "A_s_per_cpu_token": A, "B_s_per_gpu_token": Bc, "eq2_share_from_measured_A_B": r_eq2,
        "host_threads": os.cpu_count(), "device_status": st["device_status"],
        "note": "T_cpu: wall time of ipkv_attend_cpu on its thread; T_gpu, T_merge: CUDA events on the stream; medians over the "
                "second half of the steps; the engines run concurrently per layer, the join is ipkv_merge with the CPU partial "
                "in pinned host memory"}}))


def graph_microbench():
    """A launch-bound case replayed from a CUDA graph: the stateless attention call on the small configuration's
    shape (one sequence of 4096 tokens, 32 query / 4 KV heads, d 128: 4 MB of K/V, L2-resident) issued call by call
    (host: planner, table upload, two launches) against the same call recorded once and replayed."""
    import torch
    from paper_2609_14507_b200 import binding
    dev = "cuda:0"
    torch.cuda.set_device(0)
    shape = binding.AttnShape(binding.GQA, 32, 4, 128, 128, BLOCK, 128 ** -0.5)
    n = 4096
    g = torch.Generator(device=dev); g.manual_seed(1)
    k = torch.randn((n, 4, 128), generator=g, device=dev).to(torch.bfloat16)
    v = torch.randn((n, 4, 128), generator=g, device=dev).to(torch.bfloat16)
    q = torch.randn((1, 32, 128), generator=g, device=dev).to(torch.bfloat16)
    blocks = torch.zeros((n // BLOCK) * binding.ipkv_block_bytes(shape), dtype=torch.uint8, device=dev)
    binding.ipkv_pack_blocks(shape, binding.LAYOUT_TILE, k, v, n, blocks)
    runs = [[(blocks, n)]]
    o = torch.zeros((1, 32, 128), device=dev); lse = torch.zeros((1, 32), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def call():
        binding.ipkv_attend_runs_noalloc(shape, runs, q, o, lse, 0, status)

    def timed(fn, reps):
        for _ in range(20):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record(); torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / reps

    direct_us = timed(call, 2000)
    o_direct = o.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    replay_us = timed(graph.replay, 2000)
    many = torch.cuda.CUDAGraph()                            # 32 calls per graph, as 32 layers of a step would be
    with torch.cuda.graph(many):
        for _ in range(32):
            call()
    many_us = timed(many.replay, 200) / 32
    assert torch.equal(o, o_direct) and int(status.item()) == 0
    print(json.dumps({"graph_microbench": {"shape": "1 x 4096 tokens, GQA 32/4, d 128 (4.2 MB of K/V)", "direct_call_us": direct_us,
                                           "graph_replay_us": replay_us, "graph_of_32_calls_us_per_call": many_us,
                                           "kv_tokens_per_s_direct": n / (direct_us * 1e-6), "kv_tokens_per_s_graph_of_32": n / (many_us * 1e-6)}}))


def main():
    if "--graph-microbench" in sys.argv:
        graph_microbench()
        return
    if "--h2d-microbench" in sys.argv:
        h2d_microbench()
        return
    if "--cpu-engine-microbench" in sys.argv:
        cpu_engine_microbench()
        return
    if "--umma-microbench" in sys.argv:
        # cost of small tcgen05.mma instructions (one CTA, one issuing thread): fixed cost against throughput
        from paper_2609_14507_b200 import binding
        rows = binding.ipkv_probe_umma(0, 5)
        for r in rows:
            r["cycles_per_mma"] = r["total_cycles"] / r["n_mma"]
        print(json.dumps({"umma_microbench": rows, "note": "SM clocks; K = 16 per instruction, bf16 operands from shared memory "
                          "(128-byte swizzle), fp32 accumulators in tensor memory; issue = until the commit was issued, total = until it completed"}))
        return
    if "--two-engine" in sys.argv or "--two-engine-resident" in sys.argv:
        two_engine_bench(resident="--two-engine-resident" in sys.argv)
        return
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kv-splits", type=int, default=0)
    ap.add_argument("--no-read-ceiling", action="store_true", help="skip the read-only bandwidth probe reported in roofline.read_ceiling")
    ap.add_argument("--time-every", type=int, default=53,
                    help="CUDA events around every N-th attention launch of the timed region (every launch does the same work; an event "
                         "between two kernels costs the step several microseconds, so bracketing all of them would slow what is measured)")
    ap.add_argument("--no-kernel-timing", action="store_true",
                    help="diagnostic: no CUDA events around the attention launches (the roofline object is then empty); shows what the events cost the step")
    ap.add_argument("--profile-reduce", action="store_true",
                    help="diagnostic: the kernel timed by CUDA events is the split reduce, not the attention kernel (the roofline object is then meaningless)")
    ap.add_argument("--static-schedule", action="store_true",
                    help="fixed tile assignment in the grouped-query kernel (bit-reproducible) instead of dynamic balancing")
    ap.add_argument("--force-balance", action="store_true",
                    help="dynamic balancing of the grouped-query kernel whatever the launch's length (the library switches it on from 64 tiles per CTA)")
    ap.add_argument("--separate-append", action="store_true",
                    help="ipkv_append as a call and a launch of its own instead of riding in ipkv_attend_gpu")
    ap.add_argument("--separate-merge", action="store_true",
                    help="join the CPU-side partial with a separate ipkv_merge launch instead of inside the split reduce")
    ap.add_argument("--latency", action="store_true", help="also time every step separately and report P50 / P99 / max")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="default workload only: skip the short runs of the other BASELINE configurations (other_configs in the line)")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher: this process starts the replicas itself (one process per GPU, replicas only) and waits for them
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.impl == "reference":
        run_reference(args, wl, args.workload)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_14507_b200 import binding, build
    build.build()                      # no-op when libipkv.so is up to date; raises if it cannot be built
    binding.lib()                      # fail loudly if the CUDA library is missing

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    sh, B, ctx = wl["shape"], wl["batch"], wl["ctx"]
    num0, den0 = wl["share"]
    NL, Hq, Hkv, dqk, dv = sh.n_layers, sh.n_q_heads, sh.n_kv_heads, sh.dim_qk, sh.dim_v
    lens = seq_lens(wl)
    n_cpu = sum(cpu_tokens(n, num0, den0) for n in lens) // B        # mean CPU-side tokens per sequence
    n_gpu0 = sum(lens) // B - n_cpu
    total_steps = 2 * (args.warmup + args.steps) + 8
    cache = make_cache(wl, local_rank, total_steps)
    seq_ids = binding.seq_id_array(list(range(B)))
    populate(cache, wl, dev, rank)
    g = torch.Generator(device=dev); g.manual_seed(77 + rank)
    bf = torch.bfloat16
    q = torch.randn((NL, B, Hq, dqk), generator=g, device=dev).to(bf)
    k_new = torch.randn((NL, B, Hkv, dqk), generator=g, device=dev).to(bf)
    v_new = None if sh.kind == "mla" else torch.randn((NL, B, Hkv, dv), generator=g, device=dev).to(bf)
    # CPU-side partial: synthetic values of the right shape and scale (the CPU engine is outside this path)
    o_cpu = (torch.randn((NL, B * Hq, dv), generator=g, device=dev) / max(1.0, float(n_cpu)) ** 0.5).contiguous()
    lse_cpu = (torch.randn((NL, B * Hq), generator=g, device=dev) * 0.1 + float(np.log(max(1, n_cpu)))).contiguous()
    if n_cpu == 0:
        o_cpu.zero_(); lse_cpu.fill_(float("-inf"))
    o_part = torch.zeros((B, Hq, dv), device=dev)
    lse_part = torch.zeros((B, Hq), device=dev)
    fused = not args.separate_merge
    out = torch.zeros((NL, B * Hq, dv), device=dev, dtype=torch.float32 if fused else bf)
    out_lse = torch.zeros((B * Hq,), device=dev)
    cur = torch.cuda.current_stream()
    bpt = sh.bytes_per_token

    # per-layer views once, not per call: slicing a tensor costs the host a few microseconds, which the small
    # (host-bound) configuration would otherwise pay six times per layer
    q_l = [q[l] for l in range(NL)]; k_l = [k_new[l] for l in range(NL)]
    v_l = [None if v_new is None else v_new[l] for l in range(NL)]
    out_l = [out[l] for l in range(NL)]; oc_l = [o_cpu[l] for l in range(NL)]; lc_l = [lse_cpu[l] for l in range(NL)]
    apps = [{} if args.separate_append else dict(append_k=k_l[l], append_v=v_l[l]) for l in range(NL)]

    # the fused form of a layer (append riding in the call, CPU partial folded by the reduce) with its arguments marshalled once
    calls = None
    if fused and not args.separate_append:
        calls = [cache.attend_gpu_call(l, seq_ids, q_l[l], out_l[l], out_lse, kv_splits=args.kv_splits, static_schedule=args.static_schedule, force_balance=args.force_balance,
                                       stream=cur, fold_o=oc_l[l], fold_lse=lc_l[l], **apps[l]) for l in range(NL)]

    def step():
        if calls is not None:
            for call in calls:
                call()
            return
        for layer in range(NL):
            # the append rides in the attention call (the kernel writes the new rows where it can) unless --separate-append
            if args.separate_append:
                cache.append(layer, seq_ids, k_l[layer], v_l[layer], stream=cur)
            if fused:      # the CPU-side partial is joined inside the split reduce: out = merged (O, LSE)
                cache.attend_gpu(layer, seq_ids, q_l[layer], out_l[layer], out_lse, kv_splits=args.kv_splits, static_schedule=args.static_schedule, stream=cur,
                                 fold_o=oc_l[layer], fold_lse=lc_l[layer], **apps[layer])
            else:
                cache.attend_gpu(layer, seq_ids, q_l[layer], o_part, lse_part, kv_splits=args.kv_splits, static_schedule=args.static_schedule, stream=cur, **apps[layer])
                cache.merge(B * Hq, dv, [o_part.view(B * Hq, dv), oc_l[layer]], [lse_part.view(-1), lc_l[layer]],
                            out_l[layer], out_lse, out_is_bf16=True, stream=cur)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x):
        return reduce_over_ranks(x, "max", dev)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.1)                 # nvidia-smi needs a moment before its first line
    sampler.mark()                      # the samples kept are those taken under load: warm-up, timed region, end-to-end region
    for _ in range(args.warmup):
        step()
    barrier()
    st0 = cache.get_stats()
    # short runs bracket more of their launches, so that at least a dozen are timed
    args.time_every = max(1, min(args.time_every, args.steps * sh.n_layers // 12))
    cache.profile_enable(not args.no_kernel_timing, reduce=args.profile_reduce, every=args.time_every)
    cache.profile_read()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # One event per step gives medians and tails.  An event between two launches keeps the second from starting under the
    # first one's tail, which a step of a few hundred microseconds does not notice; a step of a dozen (the small L2-resident
    # case: 12 us back to back, 18 with a mark per step) is timed without them unless --latency asks for the distribution.
    step_bytes_static = sum(n - cpu_tokens(n, num0, den0) + 1 for n in lens) * bpt * NL
    with_marks = args.latency or step_bytes_static > 2 * (126 << 20)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)] if with_marks else []
    e0.record()
    for i in range(args.steps):
        if marks:
            marks[i].record()
        step()
    if marks:
        marks[-1].record()
    e1.record()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1))
    raw = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)] if marks else [ms / args.steps]
    lat = sorted(raw)
    step_ms = {"median": lat[len(lat) // 2], "best": lat[0]} if marks else {"median": None, "best": None, "note": "no per-step events on a step this short"}
    step_lat = None
    if args.latency:
        slowest = sorted(range(args.steps), key=lambda i: -raw[i])[:4]
        p99 = lat[min(len(lat) - 1, int(0.99 * len(lat)))]
        step_lat = {"p50_ms": lat[len(lat) // 2], "p99_ms": p99, "max_ms": lat[-1], "p99_over_p50": p99 / lat[len(lat) // 2],
                    "slowest_steps": [(i, round(raw[i], 3)) for i in slowest]}
    kern_ms, n_timed, n_launch = cache.profile_read()
    cache.profile_enable(False)
    st1 = cache.get_stats()
    bytes_attended = st1["kv_bytes_attended"] - st0["kv_bytes_attended"]
    h2d_stream = st1["h2d_bytes"] - st0["h2d_bytes"]
    tokens = bytes_attended // bpt
    launches = sum(st1[k] - st0[k] for k in ("attend_kernels", "reduce_kernels", "merge_kernels", "append_kernels", "pack_kernels"))
    tokens_all = reduce_over_ranks(tokens, "sum", dev)              # every replica's work, slowest replica's time
    bytes_all = reduce_over_ranks(bytes_attended, "sum", dev)
    value = tokens_all / (ms * 1e-3)
    peak, peak_kind = measured_peaks()
    ach = (bytes_attended * (n_timed / max(1, n_launch))) / (kern_ms * 1e-3) / 1e9 if kern_ms > 0 else 0.0
    roofline = {"bound": "hbm", "kernel": "attn_gqa_kernel" if sh.kind == "gqa" else "attn_mla_kernel", "achieved": ach,
                "peak": peak, "peak_kind": peak_kind + " copy bandwidth (MEASURED_PEAKS.json hbm_gbs)" if peak_kind == "measured"
                else "fallback 6650 GB/s", "unit": "GB/s", "frac": ach / peak, "frac_of_8000_nominal": ach / 8000.0,
                "avg_launch_us": 1e3 * kern_ms / max(1, n_timed), "bytes_per_launch": bytes_attended / max(1, n_launch),
                "traffic": None, "whole_step_gbs": bytes_all / (ms * 1e-3) / 1e9}
    roofline["traffic"] = DRAM_TRAFFIC_PER_LAUNCH.get(args.workload)
    if rank == 0 and world == 1 and not args.no_read_ceiling:
        # context for the fraction above: what a pure read of one launch's bytes through the same copy ring reaches
        try:
            torch.cuda.synchronize()
            best, mean = binding.ipkv_probe_read_bandwidth(local_rank, max(256 << 20, int(bytes_attended / max(1, n_launch))), 10)
            roofline["read_ceiling"] = {"best": best, "mean": mean, "unit": "GB/s", "frac_of_best": ach / best if best > 0 else None,
                                        "what": "read-only stream through the kernels' copy ring, no arithmetic, same bytes as one launch"}
        except binding.IpkvError as e:                    # e.g. no memory left for the probe's buffers
            roofline["read_ceiling"] = {"error": str(e)}

    # ---- end to end: host buffers in, host buffer out, through the same calls ---------------------------------
    e2e = None
    if not args.no_e2e:
        # One step's inputs for all layers sit in pinned host memory (queries, new K/V tokens, the CPU engine's partials);
        # each step copies them to the device, runs the path, and reads all layers' outputs back.
        hq = q.cpu().pin_memory(); hk = k_new.cpu().pin_memory()
        hv = None if v_new is None else v_new.cpu().pin_memory()
        hoc = o_cpu.cpu().pin_memory(); hlc = lse_cpu.cpu().pin_memory()
        hout = torch.zeros((NL, B * Hq, dv), dtype=out.dtype).pin_memory()
        dq = torch.empty_like(q); dk = torch.empty_like(k_new); dvn = None if v_new is None else torch.empty_like(v_new)
        doc = torch.empty_like(o_cpu); dlc = torch.empty_like(lse_cpu)

        # The copies run on a stream of their own, in groups of layers: the layers of a group start as soon as the
        # group's inputs have landed, so only the first group's copies and the last group's read-back are not hidden
        # behind the other groups' kernels, the way a server overlaps its transfers with the previous layers' work.
        # Those two groups are therefore small (one layer in front, two at the end).
        cs = torch.cuda.Stream()
        bounds = sorted({0, min(1, NL), min(4, NL), max(NL // 2, min(4, NL)), max(NL - 2, NL // 2), NL})
        n_groups = len(bounds) - 1
        landed = [torch.cuda.Event() for _ in range(n_groups)]
        computed = [torch.cuda.Event() for _ in range(n_groups)]
        step_done = torch.cuda.Event()

        def copy_in(g):
            lo, hi = bounds[g], bounds[g + 1]
            with torch.cuda.stream(cs):
                dq[lo:hi].copy_(hq[lo:hi], non_blocking=True)
                dk[lo:hi].copy_(hk[lo:hi], non_blocking=True)
                if dvn is not None:
                    dvn[lo:hi].copy_(hv[lo:hi], non_blocking=True)
                doc[lo:hi].copy_(hoc[lo:hi], non_blocking=True)
                dlc[lo:hi].copy_(hlc[lo:hi], non_blocking=True)
                landed[g].record(cs)

        dq_l = [dq[l] for l in range(NL)]; dk_l = [dk[l] for l in range(NL)]
        dv_l = [None if dvn is None else dvn[l] for l in range(NL)]
        doc_l = [doc[l] for l in range(NL)]; dlc_l = [dlc[l] for l in range(NL)]
        dapps = [{} if args.separate_append else dict(append_k=dk_l[l], append_v=dv_l[l]) for l in range(NL)]

        def run_layer(layer):
            if args.separate_append:
                cache.append(layer, seq_ids, dk_l[layer], dv_l[layer], stream=cur)
            if fused:
                cache.attend_gpu(layer, seq_ids, dq_l[layer], out_l[layer], out_lse, kv_splits=args.kv_splits, static_schedule=args.static_schedule, stream=cur,
                                 fold_o=doc_l[layer], fold_lse=dlc_l[layer], **dapps[layer])
            else:
                cache.attend_gpu(layer, seq_ids, dq_l[layer], o_part, lse_part, kv_splits=args.kv_splits, static_schedule=args.static_schedule, stream=cur, **dapps[layer])
                cache.merge(B * Hq, dv, [o_part.view(B * Hq, dv), doc_l[layer]], [lse_part.view(-1), dlc_l[layer]],
                            out_l[layer], out_lse, out_is_bf16=True, stream=cur)

        def step_e2e():
            cs.wait_event(step_done)                     # the previous step's kernels no longer read the input buffers
            copy_in(0)
            for g in range(n_groups):
                cur.wait_event(landed[g])
                run_layer(bounds[g])
                if g + 1 < n_groups:
                    copy_in(g + 1)                       # issued once this group has a kernel queued: the device never waits for the host here
                for layer in range(bounds[g] + 1, bounds[g + 1]):
                    run_layer(layer)
                computed[g].record(cur)
                with torch.cuda.stream(cs):
                    cs.wait_event(computed[g])
                    hout[bounds[g]:bounds[g + 1]].copy_(out[bounds[g]:bounds[g + 1]], non_blocking=True)
            step_done.record(cur)
            torch.cuda.synchronize()                     # the step's result is on the host

        for _ in range(args.warmup):
            step_e2e()
        barrier()
        s0 = cache.get_stats()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(args.steps):
            step_e2e()
        t1.record()
        barrier()
        ms2 = max_over_ranks(t0.elapsed_time(t1))
        s1 = cache.get_stats()
        tok2 = (s1["kv_bytes_attended"] - s0["kv_bytes_attended"]) // bpt
        h2d = NL * (hq[0].numel() * 2 + hk[0].numel() * 2 + (0 if hv is None else hv[0].numel() * 2) + hoc[0].numel() * 4 + hlc[0].numel() * 4)
        e2e = {"value": reduce_over_ranks(tok2, "sum", dev) / (ms2 * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": NL * hout[0].numel() * hout.element_size(), "ms_per_step": ms2 / args.steps}
    clocks = sampler.stop() if rank == 0 else None
    status = cache.get_stats()["device_status"]
    if status != 0:
        raise RuntimeError("a kernel reported a timed-out wait; the numbers are invalid")

    cpu = None
    others = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cache.close()
        torch.cuda.empty_cache()
        cpu = oracle_sample(wl)
    if rank == 0 and world == 1 and args.workload == DEFAULT_WORKLOAD and not args.no_other_configs:
        cache.close()                   # the other workloads need the device memory
        torch.cuda.empty_cache()
        others = [other_config(name) for name in OTHER_CONFIGS]
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_config(args.workload, wl),
            "run": {"kv_splits": args.kv_splits, "kernel_timing": "CUDA events around every %d%s attention launch" % (args.time_every, "th" if 10 <= args.time_every % 100 <= 20 else {1: "st", 2: "nd", 3: "rd"}.get(args.time_every % 10, "th")), "schedule": "static" if args.static_schedule else "dynamic balancing (GQA kernel, launches long enough for it to pay: from 64 tiles per CTA)",
                    "merge": "inside the split reduce" if fused else "separate ipkv_merge launch",
                    "append": "separate ipkv_append" if args.separate_append else "inside ipkv_attend_gpu (written by the attention kernel for GQA)",
                    "launch_overlap": "programmatic dependent launch; %d of %d attention launches started their copies before the previous kernel had completed"
                                      % (st1["early_launches"] - st0["early_launches"], st1["attend_kernels"] - st0["attend_kernels"])},
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu,
            "step_gbs": bytes_all / (ms * 1e-3) / 1e9, "step_ms": step_ms,
        }
        if step_lat:
            line["step_latency"] = step_lat
        if others is not None:
            line["other_configs"] = others
        if wl.get("grow_p"):
            line["p_growth"] = {k: st1[k] for k in ("p_segments", "p_pinned_bytes", "p_pin_us", "p_grow_waits", "p_grow_wait_us",
                                                       "p_register_us", "p_register_calls", "p_register_max_us")}
            line["p_growth"]["segments_pinned_in_timed_region"] = st1["p_segments"] - st0["p_segments"]
            line["p_growth"]["pin_ms_per_mb"] = (st1["p_pin_us"] / 1e3) / max(1.0, st1["p_pinned_bytes"] / 1e6)
        if "stream_pct" in wl:
            # the box's pinned host-to-device plateau, measured here with a 256 MB copy (best of 10 after 2 warm-ups)
            hp = torch.empty(256 << 20, dtype=torch.uint8).pin_memory(); dp = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
            best = 1e9
            for it in range(12):                                      # two untimed copies first: the first touches fault pages in
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); dp.copy_(hp, non_blocking=True); b.record(); torch.cuda.synchronize()
                if it >= 2:
                    best = min(best, a.elapsed_time(b))
            plateau = (256 << 20) / (best * 1e-3) / 1e9
            # on shared hosts the probe sometimes reads less than the streamed path just sustained: the plateau is at least that
            plateau = max(plateau, h2d_stream / (ms * 1e-3) / 1e9)
            t_h2d_ideal = h2d_stream / (plateau * 1e9) * 1e3          # ms over the timed region
            line["streaming"] = {"h2d_bytes_per_step": h2d_stream / args.steps, "h2d_gbs": h2d_stream / (ms * 1e-3) / 1e9,
                                 "h2d_plateau_gbs": plateau, "attn_kernel_ms_per_step": kern_ms / args.steps,
                                 "overlap_efficiency": max(t_h2d_ideal, kern_ms) / ms,
                                 "streamed_pct_of_p_share": wl["stream_pct"], "chunk_tokens": wl.get("chunk_tokens", 512)}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
