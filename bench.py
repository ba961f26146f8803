#!/usr/bin/env python
"""Benchmark of the KV-CAR decode hot path on B200.

One "step" = one decode step of the whole stack: for every layer, encoder +
append of the new token's K/V, then decoder + attention over the latent cache
(cached tokens restored, current token exact); then the sequence lengths advance.
Metric: decode tokens/s (sequences x steps / time), whole job.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5] [--batch B]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

Inputs are seeded and synthetic (N(0,1) K/V/Q, Xavier-uniform autoencoders, seeded
reuse map) with the shapes of the paper's GPT-2 and TinyLLaMA workloads.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import kvcar_synth as synth  # noqa: E402

METRIC = "decode tokens/s over latent KV cache"
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=12)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c5", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--batch", type=int, default=None,
                    help="override the batch (config 5 is the batch sweep; its default here is the largest point, 256)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "generic", "tensor"])
    ap.add_argument("--uncompressed", action="store_true", help="raw K/V pages (the uncompressed twin)")
    ap.add_argument("--absorbed", action="store_true",
                    help="pass KVCAR_ABSORBED: K scores from the hidden vectors (absorbed last decoder layer); the roofline "
                         "then counts that form's own, smaller number of operations")
    ap.add_argument("--absorbed-v", action="store_true",
                    help="with --absorbed: KVCAR_ABSORBED_V as well (the V side through the hidden vectors too)")
    ap.add_argument("--api", default="fused", choices=["fused", "split"],
                    help="a layer's step through kvcar_step_layer (one call; the tile kernel runs beside the encoder) "
                         "or through kvcar_encode_append + kvcar_decode_attention")
    ap.add_argument("--head-l1", action="store_true",
                    help="instead of the decode step: time Alg. 2's head-distance reduction on K rows shaped like "
                         "the workload (layers x batch*cached_tokens x KV width) and print its own JSON line")
    ap.add_argument("--prefill", action="store_true",
                    help="instead of the decode step: time the bulk encoder + append of 1024 tokens per sequence, on the "
                         "tensor cores (kvcar_encode_append_tensor) and on the CUDA cores, and print its own JSON line")
    ap.add_argument("--capacity", action="store_true",
                    help="instead of the decode step: longest sequence that fits per batch size at 0/25/50/75 %% compression from the\n"
                         "library's own bytes-per-token accounting, plus one batch actually held in memory compressed vs raw")
    ap.add_argument("--no-sweep", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="budget of the oracle sample")
    return ap.parse_args()


def workload_of(args) -> synth.Workload:
    w = synth.CONFIGS[args.workload]
    batch = args.batch or (256 if args.workload == "c5" else None)
    if batch:
        w = synth.with_batch(w, batch)
    return w


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------
def max_over_ranks(x: float, world: int, device) -> float:
    """The slowest rank's figure (replicas run independently; the job is as slow as its slowest replica)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(batch_per_rank: int, steps: int, world: int, seconds: float) -> float:
    """Replicas only (weak scaling): every rank decodes its own batch; value = all ranks' tokens / slowest time."""
    return world * batch_per_rank * steps / seconds


# ----------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.first = 0

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "5", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            t0 = time.perf_counter()      # nvidia-smi takes a moment to come up: wait for its first sample
            while not self.lines and time.perf_counter() - t0 < 3.0:
                time.sleep(0.01)
        except Exception:
            self.proc = None
        self.first = len(self.lines)      # samples before this one were taken on an idle GPU

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        lines = self.lines[self.first:] or self.lines
        for ln in lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------
def build_session(w: synth.Workload, args, torch, extra_steps: int):
    from paper_2512_06727_b200 import binding as B
    from paper_2512_06727_b200.session import Session
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    aes = {} if args.uncompressed else synth.make_stack_autoencoders(w, src, src)
    total = w.cached_tokens + extra_steps
    pps = (total + w.page_tokens - 1) // w.page_tokens
    kernel = {"auto": B.KERNEL_AUTO, "generic": B.KERNEL_GENERIC, "tensor": B.KERNEL_TENSOR}[args.kernel]
    s = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, w.batch, w.batch * pps, pps,
                w.storage, src, src, aes, kernel=kernel)
    return s, src, aes


def prefill(sess, w, torch, keep_seqs=()):
    """Fill the cache with w.cached_tokens tokens per sequence from the seeded
    device generator; returns the raw rows of `keep_seqs` (host, for the oracle)."""
    seqs = list(range(w.batch))
    for q in seqs:
        sess.ctx.seq_open(q)
    g = torch.Generator(device=sess.device)
    g.manual_seed(w.seed)
    kept = {}
    chunk = max(64, min(w.cached_tokens, (1 << 28) // max(1, w.batch * w.kv_width)))  # <= 256 Mi elements per tensor
    chunk = (chunk // w.page_tokens) * w.page_tokens or w.page_tokens
    t = 0
    while t < w.cached_tokens:
        n = min(chunk, w.cached_tokens - t)
        for l in range(w.n_layers):
            k = torch.randn(w.batch, n, w.kv_width, generator=g, device=sess.device, dtype=torch.float32).to(sess.dtype)
            v = torch.randn(w.batch, n, w.kv_width, generator=g, device=sess.device, dtype=torch.float32).to(sess.dtype)
            sess.ctx.encode_append(l, seqs, n, k.data_ptr(), v.data_ptr(), sess.stream())
            for q in keep_seqs:
                kept.setdefault((l, q), []).append((k[q].float().cpu().numpy(), v[q].float().cpu().numpy()))
            torch.cuda.current_stream().synchronize()
        sess.ctx.advance(seqs, n, sess.stream())
        t += n
    sess.ctx.sync_status(sess.stream())
    return kept


def step_inputs(sess, w, torch, n_steps):
    g = torch.Generator(device=sess.device)
    g.manual_seed(w.seed + 1000)
    k = torch.randn(n_steps, w.n_layers, w.batch, w.kv_width, generator=g, device=sess.device).to(sess.dtype)
    v = torch.randn(n_steps, w.n_layers, w.batch, w.kv_width, generator=g, device=sess.device).to(sess.dtype)
    q = torch.randn(n_steps, w.n_layers, w.batch, w.n_q_heads, w.head_dim, generator=g, device=sess.device).to(sess.dtype)
    out = torch.empty_like(q)
    return k, v, q, out


def run_step(sess, w, seqs, k, v, q, out, i, stream, flags, fused=True):
    ctx = sess.ctx
    for l in range(w.n_layers):
        if fused:
            ctx.step_layer(l, seqs, k[i, l].data_ptr(), v[i, l].data_ptr(), q[i, l].data_ptr(), out[i, l].data_ptr(),
                           flags, stream)
        else:
            ctx.encode_append(l, seqs, 1, k[i, l].data_ptr(), v[i, l].data_ptr(), stream)
            ctx.decode_attention(l, seqs, q[i, l].data_ptr(), out[i, l].data_ptr(), flags, stream)
    ctx.advance(seqs, 1, stream)


def work_per_step(sess, w, cached_tokens):
    """Algorithmic bytes / flops of the decode-attention kernels of one step."""
    by = fl = 0.0
    for l in range(w.n_layers):
        b, f = sess.ctx.layer_work_per_token(l)
        by += b * cached_tokens * w.batch
        fl += f * cached_tokens * w.batch
    return by, fl


# ----------------------------------------------------------------------------
def oracle_sample(w, src, aes, kept, steps_k, steps_v, steps_q, budget_s, gpu_out=None):
    """Time the CPU oracle as it stands on (sequence, layer) pairs of this
    workload.  Returns tokens/s scaled to the whole batch and stack, plus the
    largest deviation of the GPU outputs on the sampled pairs (if given)."""
    from oracle.kvcar_oracle import KVCAROracle
    seqs = sorted({q for (_, q) in kept})
    pps = (w.cached_tokens + 4 + w.page_tokens - 1) // w.page_tokens
    o = KVCAROracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, max(seqs) + 1,
                    len(seqs) * pps, w.storage)
    o.set_reuse_map(src, src)
    for (l, which), ae in aes.items():
        o.set_autoencoder(l, which, ae)
    for q in seqs:
        o.seq_open(q)
    # untimed: fill the oracle's own cache from the same raw rows
    n_chunks = len(kept[(0, seqs[0])])
    for c in range(n_chunks):
        n = kept[(0, seqs[0])][c][0].shape[0]
        for l in range(w.n_layers):
            k = np.stack([kept[(l, q)][c][0] for q in seqs])
            v = np.stack([kept[(l, q)][c][1] for q in seqs])
            o.encode_append(l, seqs, n, k, v)
        o.advance(seqs, n)
    # timed: decode step 0 on the sampled pairs, stopping when the budget is spent
    t0 = time.perf_counter()
    pairs = 0
    worst = 0.0
    for rep_i in range(8):       # the same step again (appending at an unadvanced position overwrites) until the budget is spent
        for q in seqs:
            for l in range(w.n_layers):
                o.encode_append(l, [q], 1, steps_k[l][q][None, None], steps_v[l][q][None, None])
                ref = o.decode_attention(l, [q], steps_q[l][q][None])
                pairs += 1
                if gpu_out is not None:
                    worst = max(worst, float(np.max(np.abs(gpu_out[l][q] - ref[0]))))
            if time.perf_counter() - t0 > budget_s:
                break
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    per_pair = dt / pairs
    step_time = per_pair * w.batch * w.n_layers
    return {"value": w.batch / step_time, "pairs": pairs, "seconds": dt, "max_abs_err_vs_gpu": worst}


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


# ----------------------------------------------------------------------------
def run_reference(args):
    """The CPU oracle as the reference arm: each step is a bounded sample of
    (sequence, layer) pairs of the workload, scaled to the whole batch."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload_of(args)
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    aes = synth.make_stack_autoencoders(w, src, src)
    from oracle.kvcar_oracle import KVCAROracle
    pps = (w.cached_tokens + args.steps + args.warmup + w.page_tokens) // w.page_tokens
    o = KVCAROracle(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, 1, pps, w.storage)
    o.set_reuse_map(src, src)
    for (l, which), ae in aes.items():
        o.set_autoencoder(l, which, ae)
    o.seq_open(0)
    rng = np.random.default_rng(w.seed)
    blk = 1024
    t = 0
    while t < w.cached_tokens:
        n = min(blk, w.cached_tokens - t)
        for l in range(w.n_layers):
            k = synth.on_grid(rng.standard_normal((1, n, w.kv_width), dtype=np.float32), w.storage)
            v = synth.on_grid(rng.standard_normal((1, n, w.kv_width), dtype=np.float32), w.storage)
            o.encode_append(l, [0], n, k, v)
        o.advance([0], n)
        t += n
    # sample: `sample_layers` layers of one sequence per step, scaled by batch * n_layers / sample_layers
    probe_layers = list(range(w.n_layers))
    times = []
    sample_layers = None
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        done = 0
        for l in probe_layers:
            k = synth.on_grid(rng.standard_normal((1, 1, w.kv_width), dtype=np.float32), w.storage)
            v = synth.on_grid(rng.standard_normal((1, 1, w.kv_width), dtype=np.float32), w.storage)
            q = synth.on_grid(rng.standard_normal((1, w.n_q_heads, w.head_dim), dtype=np.float32), w.storage)
            o.encode_append(l, [0], 1, k, v)
            o.decode_attention(l, [0], q)
            done += 1
            if sample_layers is None and time.perf_counter() - t0 > 120.0 / (args.warmup + args.steps):
                break
        if sample_layers is None:
            sample_layers = done
            probe_layers = probe_layers[:done]
        dt = time.perf_counter() - t0
        if done == w.n_layers:
            o.advance([0], 1)
        if i >= args.warmup:
            times.append(dt * w.batch * w.n_layers / done)
    ms = 1e3 * float(np.mean(times))
    value = w.batch / (ms / 1e3)
    cores = host_threads()
    sample = (f"per step: encode-append + decode attention of {sample_layers} of {w.n_layers} layers for 1 of "
              f"{w.batch} sequences at {w.cached_tokens} cached tokens, scaled by the pair count")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": w.batch, "cached_tokens": w.cached_tokens,
                       "layers": w.n_layers, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads,
                       "latent_full": w.latent_full, "reuse_frac": w.reuse_frac, "page_tokens": w.page_tokens,
                       "storage": w.storage},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------
def run_head_l1(args):
    """Alg. 2's statistic as a streaming reduction: GB/s of activations read against the measured copy bandwidth."""
    import torch
    from oracle import kvcar_oracle as orc
    from paper_2512_06727_b200 import binding as B
    w = workload_of(args)
    n_rows = w.batch * w.cached_tokens
    hkv, hd, L = w.n_kv_heads, w.head_dim, w.n_layers
    g = torch.Generator(device="cuda").manual_seed(w.seed)
    x = torch.empty(L, n_rows, hkv * hd, dtype=torch.bfloat16, device="cuda")
    x[0] = torch.randn(n_rows, hkv * hd, generator=g, device="cuda")
    for l in range(1, L):
        x[l] = x[l - 1].float() + 0.3 * torch.randn(n_rows, hkv * hd, generator=g, device="cuda")
    nbytes = B.head_l1_scratch_bytes(L, hkv, n_rows)
    scratch = torch.empty(nbytes // 4 + 4, device="cuda")
    dist_ = torch.empty(L - 1, hkv, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    K_, W_ = args.steps, max(args.warmup, 3)
    ev = []
    for i in range(W_ + K_):
        flush.fill_(i & 0xFF)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        B.head_l1_distance(L, hkv, hd, B.BF16, x.data_ptr(), n_rows, scratch.data_ptr(), nbytes, dist_.data_ptr(), stream)
        b.record()
        if i >= W_:
            ev.append((a, b))
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in ev) / len(ev)
    byts = float(x.numel() * 2)
    peaks = measured_peaks()
    gbs = byts / (ms / 1e3) / 1e9
    # parity on a sample of rows the oracle does in a moment (the rows' share of every sum is the same reduction)
    rows = min(n_rows, 256)
    sub = x[:, :rows].contiguous()
    B.head_l1_distance(L, hkv, hd, B.BF16, sub.data_ptr(), rows, scratch.data_ptr(), nbytes, dist_.data_ptr(), stream)
    torch.cuda.synchronize()
    want = orc.head_l1_distance(sub.float().cpu().numpy().astype("float64"), hkv)
    err = float(abs(dist_.cpu().numpy() - want).max() / want.max())
    print(json.dumps({"metric": "head L1 distance (Alg. 2) activations read", "value": gbs, "unit": "GB/s", "n_gpus": 1,
                      "steps": K_, "warmup": W_, "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16",
                      "data": "synthetic", "config": {"workload": w.name + "_head_l1", "layers": L, "rows": n_rows,
                                                       "kv_width": hkv * hd, "l2": "flushed between launches"},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
                                   "algorithmic_bytes_per_launch": byts},
                      "max_rel_err_vs_oracle_on_256_rows": err, "gpu_launches": 2 * K_}))


def run_capacity(args):
    """The B200 counterpart of the paper's Fig. 2 / Fig. 3 (Sec. "System Evaluation"): how long a sequence fits per
    batch size at 0 / 25 / 50 / 75 % cache compression, from the library's own bytes-per-token accounting, and one
    batch at 4096 tokens actually held in device memory, compressed (autoencoder 2x + the workload's reuse map) and raw."""
    import torch
    from paper_2512_06727_b200 import binding as B
    free_b, total_b = torch.cuda.mem_get_info()
    budget = int(free_b * 0.85)          # leave room for q/k/v, weights and the framework
    out = {"metric": "longest sequence that fits (tokens) per batch size", "unit": "tokens", "data": "accounting",
           "device_free_bytes": free_b, "device_total_bytes": total_b, "budget_bytes": budget, "curves": [], "held": []}

    def bytes_per_token(w, level):
        """level: fraction of the cache removed by autoencoders alone (no reuse), Table 2 style."""
        ctx = B.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, 1, 1, 1,
                        B.BF16 if w.storage == "bf16" else B.F32)
        none = np.full(w.n_layers * w.n_kv_heads, -1, dtype=np.int32)
        ctx.set_reuse_map(none, none)
        if level > 0:
            # 25 %: latent = half the width in half the layers; 50 %: in all layers; 75 %: a quarter of the width in all
            layers = range(w.n_layers // 2) if level == 0.25 else range(w.n_layers)
            lat_per_head = w.head_dim // 4 if level == 0.75 else w.head_dim // 2
            for l in layers:
                for which in (0, 1):
                    in_dim, hidden, latent = synth.ae_dims(w.n_kv_heads, w.head_dim, lat_per_head)
                    ctx.set_autoencoder(l, which, synth.make_autoencoder(in_dim, hidden, latent, w.seed, l, which,
                                                                         storage=w.storage))
        comp, full = ctx.cache_bytes_per_token()
        return comp, full

    for name in ("c5", "c3"):
        w = synth.CONFIGS[name]
        for level in (0.0, 0.25, 0.5, 0.75):
            comp, full = bytes_per_token(w, level)
            row = {"shape": "GPT-2-small 12x12x64" if name == "c5" else "TinyLLaMA 22 layers, 4 KV heads x 64",
                   "compression": level, "cache_bytes_per_token": comp, "saved": 1.0 - comp / full, "max_tokens": {}}
            for b in (1, 8, 16, 32, 64, 128, 256):
                row["max_tokens"][str(b)] = int(budget // (b * comp))
            out["curves"].append(row)

    # one batch at 4096 tokens held for real: the workload's own configuration (autoencoders + reuse map) and its raw twin
    w = synth.CONFIGS["c5"]
    from paper_2512_06727_b200.session import Session
    src = synth.make_reuse_map(w.n_layers, w.n_kv_heads, w.reuse_frac, w.seed)
    pps = (w.cached_tokens + 1 + w.page_tokens - 1) // w.page_tokens
    for label, aes in (("compressed", synth.make_stack_autoencoders(w, src, src)), ("raw", {})):
        probe = B.Context(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, 1, 1, 1, B.BF16)
        probe.set_reuse_map(src, src)
        for (l, which), ae in aes.items():
            probe.set_autoencoder(l, which, ae)
        comp, full = probe.cache_bytes_per_token()
        n_seq = int(budget // (comp * pps * w.page_tokens))
        torch.cuda.empty_cache()
        sess = Session(w.n_layers, w.n_q_heads, w.n_kv_heads, w.head_dim, w.page_tokens, n_seq, n_seq * pps, pps,
                       w.storage, src, src, aes)
        allseq = list(range(n_seq))
        for q_ in allseq:
            sess.ctx.seq_open(q_)
        for i in range(0, n_seq, B.MAX_BATCH):       # pages for every sequence; the rows keep the pool's zeros
            part = allseq[i:i + B.MAX_BATCH]
            sess.ctx.reserve(part, w.cached_tokens)
            sess.ctx.advance(part, w.cached_tokens, sess.stream())
        last = allseq[-min(B.MAX_BATCH, n_seq):]
        k = torch.randn(len(last), w.kv_width, device="cuda").to(sess.dtype)
        q = torch.randn(len(last), w.n_q_heads, w.head_dim, device="cuda").to(sess.dtype)
        o = torch.empty_like(q)
        t0 = time.perf_counter()
        for l in range(w.n_layers):                  # one decode step over the last sequences of the pool
            sess.ctx.step_layer(l, last, k.data_ptr(), k.data_ptr(), q.data_ptr(), o.data_ptr(), B.INCLUDE_CURRENT_EXACT,
                                sess.stream())
        sess.ctx.sync_status(sess.stream())
        dt = time.perf_counter() - t0
        out["held"].append({"layout": label, "cached_tokens": w.cached_tokens, "sequences_held": n_seq,
                            "pool_bytes": sess.sizes[0], "cache_bytes_per_token": comp,
                            "decode_step_of_last_sequences": {"sequences": len(last), "seconds": dt,
                                                              "finite": bool(torch.isfinite(o.float()).all().item())}})
        del sess
        torch.cuda.empty_cache()
    print(json.dumps(out))


def run_prefill(args):
    """Bulk encoder + append: one call per layer of 1024 new tokens per sequence."""
    import torch
    w = workload_of(args)
    chunk = 1024
    K_, W_ = args.steps, max(args.warmup, 3)
    peaks = measured_peaks()
    out = {}
    for name in ("tensor", "cuda_cores"):
        sess, src, aes = build_session(synth.scaled(w, cached_tokens=0), args, torch, chunk * (K_ + W_) + 8)
        seqs = list(range(w.batch))
        for q in seqs:
            sess.ctx.seq_open(q)
        g = torch.Generator(device="cuda").manual_seed(w.seed)
        k = torch.randn(w.batch, chunk, w.kv_width, generator=g, device="cuda").to(torch.bfloat16)
        v = torch.randn(w.batch, chunk, w.kv_width, generator=g, device="cuda").to(torch.bfloat16)
        stream = sess.stream()
        call = sess.ctx.encode_append_tensor if name == "tensor" else sess.ctx.encode_append
        ms = []
        for i in range(W_ + K_):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for l in range(w.n_layers):
                call(l, seqs, chunk, k.data_ptr(), v.data_ptr(), stream)
            b.record()
            sess.ctx.advance(seqs, chunk, stream)
            torch.cuda.synchronize()
            if i >= W_:
                ms.append(a.elapsed_time(b))
        sess.ctx.sync_status(stream)
        out[name] = sum(ms) / len(ms)
        flops = 0.0
        for (l, which), ae in aes.items():
            flops += 2.0 * (ae["in_dim"] * ae["hidden"] + ae["hidden"] * ae["latent"]) * w.batch * chunk
        del sess
    tf = flops / (out["tensor"] / 1e3) / 1e12
    print(json.dumps({"metric": "prefill tokens/s (bulk encoder + append, all layers)", "value": w.batch * chunk / (out["tensor"] / 1e3),
                      "unit": "tokens/s", "n_gpus": 1, "steps": K_, "warmup": W_, "ms_per_step": out["tensor"],
                      "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": w.name + "_prefill", "layers": w.n_layers, "rows_per_call": w.batch * chunk},
                      "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                   "frac": tf / peaks["bf16_tflops"], "traffic": None, "peak_source": peaks["source"] + " (burst)",
                                   "algorithmic_flops_per_step": flops},
                      "cuda_core_encoder_ms_per_step": out["cuda_cores"]}))


NOMINAL_BF16_TFLOPS = 2250.0     # dense bf16 per B200 (vendor figure): context beside the measured peaks
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes (read + write) per decode-kernel launch and listed sequence, from an ncu capture of the GPT-2-shaped
# stack at 4096 cached tokens (batch 8, scaled by the batch: a launch's traffic is its sequences' latent rows)
NCU_TRAFFIC = {"c5": {"bytes_per_sequence": 54.23e6 / 8, "captured_on": "c5_gpt2s_12l_L4096_b8",
                      "profile": "profiles/decode_pair_kernel_c5.md"}}


def roofline_of(flops, byts, seconds, peaks, launches):
    """Both sides of the roofline for `launches` launches that took `seconds` in all: the slower of algorithmic bytes
    at the measured copy bandwidth and algorithmic flops at the measured bf16 peak is the bound; the kernel is timed
    alone (one event pair per launch), so the burst figure is the tensor peak."""
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    tensor = t_tc >= t_hbm
    ach = flops / seconds / 1e12 if tensor else byts / seconds / 1e9
    peak = peaks["bf16_tflops"] if tensor else peaks["hbm_gbs"]
    r = {"bound": "tensor" if tensor else "hbm", "achieved": ach, "peak": peak, "unit": "TFLOP/s" if tensor else "GB/s",
         "frac": max(t_hbm, t_tc) / seconds, "traffic": None,
         "peak_source": peaks["source"] + (" (burst: kernel timed alone)" if tensor else " (copy)"),
         "kernel": "decode_attention (decoder + attention + combine)", "launches": launches,
         "avg_launch_us": 1e6 * seconds / launches,
         "algorithmic_flops_per_launch": flops / launches, "algorithmic_bytes_per_launch": byts / launches,
         "tensor_side_frac": t_tc / seconds, "hbm_side_frac": t_hbm / seconds,
         "frac_of_sustained_bf16": flops / seconds / 1e12 / peaks["bf16_tflops_sustained"],
         "frac_of_nominal_bf16": flops / seconds / 1e12 / NOMINAL_BF16_TFLOPS,
         "frac_of_nominal_hbm": byts / seconds / 1e9 / NOMINAL_HBM_GBS}
    return r


def fast_prefill(sess, w, torch):
    """Untimed cache fill for the bench: the tensor-core bulk encoder where the layer has one, else the general one."""
    seqs = list(range(w.batch))
    for q in seqs:
        sess.ctx.seq_open(q)
    g = torch.Generator(device=sess.device)
    g.manual_seed(w.seed)
    chunk = max(64, min(w.cached_tokens, (1 << 27) // max(1, w.batch * w.kv_width)))
    chunk = (chunk // w.page_tokens) * w.page_tokens or w.page_tokens
    use_tensor = w.storage == "bf16" and sess.has_autoencoders
    t = 0
    while t < w.cached_tokens:
        n = min(chunk, w.cached_tokens - t)
        k = torch.randn(w.batch, n, w.kv_width, generator=g, device=sess.device, dtype=torch.float32).to(sess.dtype)
        v = torch.randn(w.batch, n, w.kv_width, generator=g, device=sess.device, dtype=torch.float32).to(sess.dtype)
        for l in range(w.n_layers):       # the same rows for every layer: content does not matter to the timing
            call = sess.ctx.encode_append_tensor if use_tensor else sess.ctx.encode_append
            call(l, seqs, n, k.data_ptr(), v.data_ptr(), sess.stream())
        torch.cuda.current_stream().synchronize()
        sess.ctx.advance(seqs, n, sess.stream())
        t += n
    sess.ctx.sync_status(sess.stream())


def measure(w, args, torch, B, steps, warmup, uncompressed, flush, peaks, fused=True, keep=False):
    """One workload: tokens/s through the per-layer step (all kernels of a step, L2 flushed between steps) and the
    decode-attention call alone per launch (L2 flushed between launches)."""
    class A: pass
    a2 = A(); a2.uncompressed = uncompressed; a2.kernel = args.kernel
    sess, src, aes = build_session(w, a2, torch, 2 * (warmup + steps) + 24)
    sess.has_autoencoders = bool(aes)
    fast_prefill(sess, w, torch)
    seqs = list(range(w.batch))
    stream = sess.stream()
    absorbed = bool(getattr(args, "absorbed", False)) and not uncompressed
    both = absorbed and bool(getattr(args, "absorbed_v", False))
    flags = B.INCLUDE_CURRENT_EXACT | (B.ABSORBED if absorbed else 0) | (B.ABSORBED_V if both else 0)
    n_in = 4
    k, v, q, out = step_inputs(sess, w, torch, n_in)       # a few input sets, cycled (values do not matter)
    for i in range(warmup):
        run_step(sess, w, seqs, k, v, q, out, i % n_in, stream, flags, fused)
    sess.ctx.sync_status(stream)
    launches0 = sess.ctx.launch_count()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    for j in range(steps):
        flush.fill_(j & 0xFF)
        ev[j][0].record()
        run_step(sess, w, seqs, k, v, q, out, j % n_in, stream, flags, fused)
        ev[j][1].record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    total_ms = float(sum(a_.elapsed_time(b_) for a_, b_ in ev))
    launches = sess.ctx.launch_count() - launches0
    sess.ctx.sync_status(stream)
    # the decode-attention call alone
    kev = []
    n_k = max(1, min(steps, 4))
    for j in range(n_k):
        L = sess.ctx.seq_len(0)
        for l in range(w.n_layers):
            sess.ctx.encode_append(l, seqs, 1, k[j % n_in, l].data_ptr(), v[j % n_in, l].data_ptr(), stream)
            flush.fill_(l & 0xFF)
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record()
            sess.ctx.decode_attention(l, seqs, q[j % n_in, l].data_ptr(), out[j % n_in, l].data_ptr(), flags, stream)
            b_.record()
            kev.append((l, L, a_, b_))
        sess.ctx.advance(seqs, 1, stream)
    torch.cuda.synchronize()
    sess.ctx.sync_status(stream)
    plain_flops = sum(sess.ctx.layer_work_per_token(l)[1] * L * w.batch for (l, L, _, _) in kev)
    flops = sum(sess.ctx.layer_work_absorbed(l, both) * L * w.batch for (l, L, _, _) in kev) if absorbed else plain_flops
    byts = sum(sess.ctx.layer_work_per_token(l)[0] * L * w.batch for (l, L, _, _) in kev)
    kern_s = sum(a_.elapsed_time(b_) for (_, _, a_, b_) in kev) / 1e3
    roof = roofline_of(flops, byts, kern_s, peaks, len(kev))
    if absorbed:   # the plain form's operations over the same time: what the absorbed form is worth as plain-form throughput
        roof["form"] = ("absorbed K and V sides (KVCAR_ABSORBED | KVCAR_ABSORBED_V)" if both else
                        "absorbed K scores (KVCAR_ABSORBED)") + ": achieved and frac count this form's own operations"
        roof["plain_form_flops_per_launch"] = plain_flops / len(kev)
        roof["plain_form_equivalent_frac"] = plain_flops / kern_s / 1e12 / roof["peak"] if roof.get("bound") == "tensor" else None
    comp, full = sess.ctx.cache_bytes_per_token()
    res = {"tokens_per_s": w.batch * steps / (total_ms / 1e3), "ms_per_step": total_ms / steps, "steps": steps,
           "roofline": roof, "cache_bytes_per_token": comp, "uncompressed_bytes_per_token": full, "launches": int(launches),
           "wall_s": wall, "total_ms": total_ms}
    if keep:
        res["session"] = (sess, src, aes, k, v, q, out)
    else:
        del sess
        torch.cuda.empty_cache()
    return res


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.prefill:
        run_prefill(args)
        return
    if args.head_l1:
        run_head_l1(args)
        return
    if args.capacity:
        run_capacity(args)
        return
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    from paper_2512_06727_b200 import binding as B

    w = workload_of(args)
    K_, W_ = args.steps, max(args.warmup, 3)
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=f"cuda:{local}")
    fused = args.api == "fused"

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the headline workload ----------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier()
    head = measure(w, args, torch, B, K_, W_, bool(args.uncompressed), flush, peaks, fused=fused, keep=True)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(head["total_ms"], world, torch.device(f"cuda:{local}"))
    ms_per_step = total_ms / K_
    value = whole_job_tokens_per_s(w.batch, K_, world, total_ms / 1e3)
    roof = head["roofline"]
    cfg_key = args.workload
    if not args.uncompressed and args.kernel == "auto" and cfg_key in NCU_TRAFFIC:
        t = NCU_TRAFFIC[cfg_key]
        roof["traffic"] = t["bytes_per_sequence"] * w.batch
        roof["traffic_source"] = (f"ncu dram__bytes_read.sum + dram__bytes_write.sum of one launch on {t['captured_on']}, "
                                  f"scaled by the batch; {t['profile']}")
    sess, src, aes, k, v, q, out = head.pop("session")
    seqs = list(range(w.batch))
    stream = sess.stream()
    flags = B.INCLUDE_CURRENT_EXACT | (B.ABSORBED if (args.absorbed and not args.uncompressed) else 0) | \
        (B.ABSORBED_V if (args.absorbed and args.absorbed_v and not args.uncompressed) else 0)

    # ---- e2e: host buffers through the C ABI, copies inside the timed region ----
    e2e = None
    n_e2e = 0 if args.no_e2e else max(2, min(K_, 6))
    if n_e2e:
        hk = [k[0, l].cpu().pin_memory() for l in range(w.n_layers)]
        hv = [v[0, l].cpu().pin_memory() for l in range(w.n_layers)]
        hq = [q[0, l].cpu().pin_memory() for l in range(w.n_layers)]
        ho = [torch.empty_like(hq[l]).pin_memory() for l in range(w.n_layers)]

        def e2e_step():
            for l in range(w.n_layers):
                sess.ctx.step_layer_host(l, seqs, hk[l].data_ptr(), hv[l].data_ptr(), hq[l].data_ptr(),
                                         ho[l].data_ptr(), flags, stream)
            sess.ctx.advance(seqs, 1, stream)
            torch.cuda.current_stream().synchronize()      # the step's result is on the host
        for _ in range(2):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        barrier()
        e2e_s = max_over_ranks(time.perf_counter() - t0, world, torch.device(f"cuda:{local}"))
        elem = 2 if w.storage == "bf16" else 4
        e2e = {"value": whole_job_tokens_per_s(w.batch, n_e2e, world, e2e_s), "unit": UNIT, "steps": n_e2e,
               "h2d_bytes_per_step": w.n_layers * w.batch * (2 * w.kv_width + w.n_q_heads * w.head_dim) * elem,
               "d2h_bytes_per_step": w.n_layers * w.batch * w.n_q_heads * w.head_dim * elem,
               "timing": "wall clock around K host-buffer steps, stream synchronised every step"}
        sess.ctx.sync_status(stream)
    del sess
    torch.cuda.empty_cache()

    # ---- CPU baseline: the oracle on a bounded sample of the headline workload ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # a small replica of the workload (same shapes and length, two sequences) filled through the general encoder,
        # whose rows the oracle mirrors; a decode step of it is compared with the oracle and the oracle is timed
        w2 = synth.with_batch(w, 2)
        class A2: pass
        a2 = A2(); a2.uncompressed = bool(args.uncompressed); a2.kernel = args.kernel
        sess2, src2, aes2 = build_session(w2, a2, torch, 4)
        kept2 = prefill(sess2, w2, torch, (0, 1))
        k2, v2, q2, out2 = step_inputs(sess2, w2, torch, 1)
        run_step(sess2, w2, [0, 1], k2, v2, q2, out2, 0, sess2.stream(), flags)
        torch.cuda.synchronize()
        sk = [k2[0, l].float().cpu().numpy() for l in range(w.n_layers)]
        sv = [v2[0, l].float().cpu().numpy() for l in range(w.n_layers)]
        sq = [q2[0, l].float().cpu().numpy() for l in range(w.n_layers)]
        go = [out2[0, l].float().cpu().numpy().astype(np.float64) for l in range(w.n_layers)]
        del sess2
        r = oracle_sample(w, src2, aes2, kept2, sk, sv, sq, args.cpu_seconds, go)
        cpu = {"value": r["value"], "unit": UNIT, "cores": host_threads(), "kind": "oracle",
               "sample": f"decode step at {w.cached_tokens} cached tokens: {r['pairs']} (sequence, layer) pair evaluations "
                         f"on two sequences of the same shapes ({r['seconds']:.1f} s), scaled to the "
                         f"{w.batch * w.n_layers} pairs of a step",
               "max_abs_err_gpu_vs_oracle_on_sample": r["max_abs_err_vs_gpu"]}

    # ---- the other configurations, shorter runs (parity cases of the test-suite, timed here for the record) ----
    configs = None
    if rank == 0 and world == 1 and not args.no_sweep:
        configs = []
        sweep = [("c1", None), ("c2", None), ("c3", None), ("c4", None)] + [("c5", b) for b in (1, 8, 32, 128, 256)]
        for name, batch in sweep:
            wc = synth.CONFIGS[name]
            if batch:
                wc = synth.with_batch(wc, batch)
            big = wc.batch * wc.cached_tokens * wc.n_layers
            st_ = 2 if big > 5e6 else 4
            row = {"workload": wc.name, "batch": wc.batch, "cached_tokens": wc.cached_tokens, "layers": wc.n_layers,
                   "dtype": wc.storage}
            try:
                if wc.name == w.name and not args.uncompressed:
                    c = head
                else:
                    c = measure(wc, args, torch, B, st_, 3, False, flush, peaks)
                r_ = c["roofline"]
                row.update({"tokens_per_s": c["tokens_per_s"], "ms_per_step": c["ms_per_step"], "steps": c["steps"],
                            "us_per_launch": r_["avg_launch_us"], "bound": r_["bound"], "frac": r_["frac"],
                            "frac_of_sustained_bf16": r_["frac_of_sustained_bf16"], "achieved": r_["achieved"],
                            "achieved_unit": r_["unit"],
                            "cache_bytes_per_token": c["cache_bytes_per_token"],
                            "uncompressed_bytes_per_token": c["uncompressed_bytes_per_token"]})
                if wc.storage == "bf16":
                    u = measure(wc, args, torch, B, st_, 3, True, flush, peaks)
                    ru = u["roofline"]
                    row["raw_twin"] = {"tokens_per_s": u["tokens_per_s"], "us_per_launch": ru["avg_launch_us"],
                                       "bound": ru["bound"], "frac": ru["frac"], "achieved_gbs": ru["achieved"],
                                       "cache_bytes_per_token": u["cache_bytes_per_token"]}
                # the headline workload once more with the K side in the absorbed form (same results up to rounding)
                if wc.name == w.name and wc.storage == "bf16" and not args.absorbed and not args.uncompressed:
                    class A2: pass
                    for key, both_ in (("absorbed_k", False), ("absorbed_kv", True)):
                        a2 = A2(); a2.kernel = args.kernel; a2.absorbed = True; a2.absorbed_v = both_
                        ab = measure(wc, a2, torch, B, st_, 3, False, flush, peaks)
                        ra = ab["roofline"]
                        row[key] = {"tokens_per_s": ab["tokens_per_s"], "us_per_launch": ra["avg_launch_us"],
                                    "frac_on_own_operation_count": ra["frac"],
                                    "frac_if_credited_with_the_plain_form": ra.get("plain_form_equivalent_frac")}
            except Exception as ex:      # a configuration that does not fit or fails is reported, not fatal
                row["error"] = str(ex)[:200]
            configs.append(row)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K_, "warmup": W_,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if w.storage == "bf16" else "f32", "data": "synthetic",
                "config": {"workload": w.name, "batch_per_gpu": w.batch, "cached_tokens": w.cached_tokens,
                           "layers": w.n_layers, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads,
                           "latent_full": 0 if args.uncompressed else w.latent_full, "reuse_frac": w.reuse_frac,
                           "page_tokens": w.page_tokens, "kernel": args.kernel, "api": args.api,
                           "uncompressed": bool(args.uncompressed), "absorbed": ("kv" if args.absorbed_v else "k") if (args.absorbed and not args.uncompressed) else False,
                           "storage": w.storage,
                           "l2": "flushed between steps and between the per-launch timings (256 MiB write outside the event pairs)",
                           "cache_bytes_per_token": head["cache_bytes_per_token"],
                           "uncompressed_bytes_per_token": head["uncompressed_bytes_per_token"],
                           "wall_s_timed_region": head["wall_s"]},
                "clocks": clocks, "roofline": roof, "cpu_baseline": cpu, "e2e": e2e,
                "gpu_launches": head["launches"], "configs": configs}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
