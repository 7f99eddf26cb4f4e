#!/usr/bin/env python
"""Benchmark of the GPU-resident serving loop on the 8B-shaped configuration.

One "step" is one iteration of the whole hot path (control plane + forward of the
composed batch + sampling + publish).  The default run

  1. builds the library, draws seeded bf16 weights on the device, carves the KV pool;
  2. times the oracle on a bounded sample on the host cores (`cpu_baseline`);
  3. closed-loop saturation run of the request stream in manual mode: a ramp that brings
     the batch to steady state, W warm-up steps, then EXACTLY K steps in one launch of the
     loop kernel, timed with CUDA events on the library's stream -> `value`, `roofline`;
  4. the same stream end to end through blink_submit / blink_poll with host buffers and
     the persistent loop -> `e2e`;
  5. a real-time Poisson run at the configuration's offered load -> `latency`
     (p50 / p99 TTFT and TPOT; `--interfere` adds a host-CPU stress process).

`--impl reference` times the CPU oracle alone on the same configuration and metric.
Under torchrun every rank runs an independent replica (the path has no exchange step);
the value is the sum over ranks divided by the slowest rank's time.
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
sys.path.insert(0, ROOT)


POLICY = 0   # BLINK_POLICY_* used by every engine this run creates (--policy)

# DRAM traffic of one step (dram__bytes_read.sum + dram__bytes_write.sum over all phases), from the ncu
# capture summarised in the named file under profiles/: the same device code launched phase by phase on a
# 4-layer model of the same layer shape, per-layer phases averaged and scaled to the full layer count.
# `algorithmic_gb` is the algorithmic figure (step_bytes_flops) of the captured step at the full layer
# count; the bench scales the traffic to its own steps by the ratio of algorithmic bytes.  `digest` is
# kernel_digest() at capture time: once the kernels change the figure is stale and is reported as null.
TRAFFIC = {
    "C3 8B stream": dict(traffic_gb=45.55, algorithmic_gb=40.596, digest="3c3e2e4e64c46518",
                         source="profiles/dram_traffic_8B_stepped.md"),
}


def kernel_digest():
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2604_07609_b200", "csrc")
    for f in ("forward.cuh", "gemm_tc.cuh", "attention.cuh", "kernels.cuh"):   # the phases that move the data
        h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def log(*a):
    print(*a, file=sys.stderr, flush=True)


# ----------------------------------------------------------------------------------------------
def model_numbers(m):
    esz = 2 if m.dtype == "bf16" else 4
    E1 = max(1, m.n_experts)
    per_layer = m.qkv_dim * m.d_model + m.d_model * m.q_dim + E1 * 3 * m.d_ff * m.d_model
    layer_params_dense_active = m.qkv_dim * m.d_model + m.d_model * m.q_dim + \
        (m.top_k_experts if m.n_experts else 1) * 3 * m.d_ff * m.d_model
    return dict(esz=esz,
                w_touched_bytes=(m.n_layers * per_layer + m.vocab * m.d_model) * esz,
                p_layers=m.n_layers * layer_params_dense_active,
                kv_bytes_per_token=m.n_layers * 2 * m.n_kv_heads * m.head_dim * esz)


def step_bytes_flops(m, st):
    """Algorithmic bytes and flops of the steps in `st` (per-iteration records):
    bytes = weights touched + KV read (each request's context once) + KV written
            + activations (~40 B per row per d) + logits written;
    flops = 2 * rows * layer params + 2 * sample rows * V * d + 4 * keys attended * Hq * hd * L."""
    nb = model_numbers(m)
    T = st["n_tokens"].astype(np.float64)
    rows = st["n_sample_rows"].astype(np.float64)
    by = nb["w_touched_bytes"] + st["kv_tokens"].astype(np.float64) * nb["kv_bytes_per_token"] + \
        T * nb["kv_bytes_per_token"] + T * m.d_model * 40.0 + rows * m.vocab * 4.0
    fl = 2.0 * T * nb["p_layers"] + 2.0 * rows * m.vocab * m.d_model + \
        4.0 * st["ctx_tokens"].astype(np.float64) * m.n_q_heads * m.head_dim * m.n_layers
    return by, fl


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], tf_burst=d["bf16_tflops"], tf_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while a region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index=0):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = f"/tmp/blink_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            p = [x.strip() for x in line.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2])); power.append(float(p[3]))
            except ValueError:
                continue
            for n, v in zip(names, p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        hi = [s for s in sm if s > 0.5 * max(sm)] or sm
        return dict(sm_mhz=float(np.median(hi)), sm_max_mhz=float(max(mx)), power_w_max=float(max(power)),
                    samples=len(sm), reasons=sorted(reasons))


# ----------------------------------------------------------------------------------------------
def weights_to_host_fp32(m, wbuf):
    """Per-tensor, per-layer copies so that no big temporary lands on the device."""
    import torch
    from synth import weight_layout
    layout, _ = weight_layout(m)
    out = {}
    for name, (off, shape, dt) in layout.items():
        n = int(np.prod(shape))
        if n == 0:
            out[name] = np.zeros(shape, dtype=np.float32)
            continue
        esz = 4 if dt == torch.float32 else 2
        host = wbuf[off:off + n * esz].cpu().view(dt)
        out[name] = host.to(torch.float32).numpy().reshape(shape)
    return out


def sample_requests(config, n_requests, prompt_cap, new_tokens):
    from synth import make_requests
    reqs = make_requests(config, n_requests=n_requests)
    for r in reqs:
        r.prompt = r.prompt[:prompt_cap]
        r.max_new = new_tokens
    return reqs


def cpu_oracle_sample(m, sched, wbuf, n_requests, prompt_cap, new_tokens, config, keep_logits=False):
    """Time the oracle, as it stands, on a bounded sample of the workload."""
    import torch
    from oracle import serve as OS
    from oracle import transformer as O2
    reqs = sample_requests(config, n_requests, prompt_cap, new_tokens)
    arrays = weights_to_host_fp32(m, wbuf)
    W = O2.Weights(m, arrays, dtype=np.float32)
    sch = sched.with_(n_blocks=max(64, n_requests * ((prompt_cap + new_tokens) // 16 + 2)))
    t0 = time.perf_counter()
    res = OS.run(m, sch, W, reqs, act_round=O2.round_bf16 if m.dtype == "bf16" else None, keep_logits=keep_logits)
    dt = time.perf_counter() - t0
    if keep_logits:   # untimed: the same sample through the plain oracle (no rounding hook), same tokens fed back
        res["plain"] = OS.run(m, sch, W, reqs, act_round=None, forced=res["tokens"]) if m.dtype == "bf16" else res
        res["requests"], res["sched"] = reqs, sch
    n_out = sum(len(v) for v in res["tokens"].values())
    return dict(value=n_out / dt, unit="output tok/s", cores=torch.get_num_threads(), kind="oracle",
                sample=f"first {n_requests} requests of the stream, prompts cut to {prompt_cap} tokens, "
                       f"{new_tokens} new tokens each, full {m.n_layers}-layer model in fp32 numpy; "
                       f"{n_out} tokens in {dt:.1f} s, {len(res['trace'])} iterations"), res, dt


def parity_on_sample(B, m, wbuf, wl, res):
    """The oracle's sample (the one the CPU leg just timed, full model) through the GPU loop, teacher-forced
    with the oracle's tokens, logits captured: how far the two are apart, beside how far the two CPU
    oracles (with and without the 16-bit rounding hook) are from each other on the same inputs."""
    import torch
    reqs, sch = res["requests"], res["sched"]
    dev = wbuf.device
    total = sum(r.max_new for r in reqs)
    kv = torch.zeros(sch.n_blocks * B.kv_bytes_per_block(m, sch.block_size), dtype=torch.uint8, device=dev)
    cap = torch.zeros((total, m.vocab), dtype=torch.float32, device=dev)
    eng = B.Blink(m, sch, wbuf, kv, start_paused=True, logits_capture=cap, idle_exit_us=300_000, weights_layout=wl,
                  trace_words=1 << 20)
    try:
        for r in reqs:
            eng.submit_request(r, forced_tokens=res["tokens"][r.ticket])
        eng.blink_start()
        ev = eng.drain(total, timeout_s=120)
        eng.blink_stop(final=False)
        trace = B.parse_trace(eng.blink_get_trace())
    finally:
        eng.blink_destroy()
    torch.cuda.synchronize()
    lg = cap.cpu().numpy().astype(np.float64)
    lo = np.stack([row for (_, _, _, _, row) in res["logits"]]).astype(np.float64)
    lp = np.stack([row for (_, _, _, _, row) in res["plain"]["logits"]]).astype(np.float64)
    rms = lambda x: float(np.sqrt(np.mean(x * x)))
    same_trace = [(r["admitted"], r["scheduled"], r["allocated"], r["finished"], r["freed"]) for r in trace] == \
                 [(r["admitted"], r["scheduled"], r["allocated"], r["finished"], r["freed"]) for r in res["trace"]]
    toks = B.tokens_by_ticket(ev)
    agree = sum(toks[t][i] == res["sampled"][t][i] for t in toks for i in range(len(toks[t])))
    return dict(rows=int(lg.shape[0]), logit_std=float(lp.std()), trace_equal=bool(same_trace),
                parity_max_abs=float(np.abs(lg - lo).max()), parity_rms=rms(lg - lo),
                vs_plain_oracle_max_abs=float(np.abs(lg - lp).max()), vs_plain_oracle_rms=rms(lg - lp),
                oracle_rounding_noise_max_abs=float(np.abs(lo - lp).max()), oracle_rounding_noise_rms=rms(lo - lp),
                sampled_tokens_equal=f"{agree}/{total}",
                note="gpu logits vs the CPU oracle on the cpu_baseline sample (full model, teacher-forced); "
                     "parity_* against the oracle with the data path's 16-bit rounding points, vs_plain_* against the "
                     "oracle without them; oracle_rounding_noise_* is the distance between those two oracles")


# ----------------------------------------------------------------------------------------------
class Stressor:
    """Host-CPU interference: one pinned process per core, half spinning on integer
    arithmetic, half streaming over arrays larger than the last-level cache."""

    def __init__(self):
        self.procs = []

    def start(self):
        code_int = "x=1\nwhile True:\n    x=(x*6364136223846793005+1442695040888963407)&0xFFFFFFFFFFFFFFFF\n"
        code_mem = ("import numpy as np\na=np.ones(1<<25);b=np.ones(1<<25);c=np.ones(1<<25)\n"
                    "while True:\n    np.add(b,c,out=a);np.multiply(a,1.0001,out=b)\n")
        n = os.cpu_count() or 1
        for i in range(n):
            code = code_int if i % 2 == 0 else code_mem
            p = subprocess.Popen([sys.executable, "-c", code], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
            try:
                os.sched_setaffinity(p.pid, {i})
            except Exception:
                pass
            self.procs.append(p)
        time.sleep(1.0)

    def stop(self):
        for p in self.procs:
            p.terminate()
        for p in self.procs:
            try:
                p.wait(timeout=5)
            except Exception:
                p.kill()
        self.procs = []


def decode_point(B, m, sched, wbuf, kv, wl, gemm_impl, n, in_len, out_len, steps, cfg_i):
    """Fixed-batch decode steps (an N x I -> O closed batch past its prefill): the clean
    bandwidth-bound operating point.  Returns ms/step and the HBM-roofline fractions."""
    from synth.workload import closed_batch
    reqs = closed_batch(n, in_len, out_len, m.vocab, seed=7, top_k=50 if cfg_i >= 3 else 0, temperature=0.8)
    ramp = (n * in_len + sched.prefill_chunk_tokens - 1) // sched.prefill_chunk_tokens + 2
    eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_MANUAL, gemm_impl=gemm_impl, stats_iters=ramp + steps + 16,
                  idle_exit_us=200_000, weights_layout=wl, policy=POLICY)
    try:
        for r in reqs:
            eng.submit_request(r)
        eng.blink_run(ramp)
        eng.blink_run(3)
        while len(eng.blink_poll(4096, 0)):
            pass
        it0 = int(eng.blink_get_stats().iterations)
        ms = eng.blink_run(steps)
        its = eng.blink_get_iter_stats()[it0:it0 + steps]
    finally:
        eng.blink_destroy()
    by, _ = step_bytes_flops(m, its)
    pk = measured_peaks()
    gbs = float(by.sum() / (ms / 1e3) / 1e9)
    return dict(batch=float(its["n_decode"].mean()), ctx_mean=float(its["kv_tokens"].mean() / max(1.0, its["n_items"].mean())),
                steps=int(len(its)), ms_per_step=ms / max(1, len(its)), algorithmic_gb_per_step=float(by.mean() / 1e9),
                achieved_gbs=gbs, frac_of_measured_hbm=gbs / pk["hbm_gbs"], frac_of_8TBs_spec=gbs / 8000.0,
                tok_s=float(its["n_sample_rows"].sum() / (ms / 1e3)))


def reduce_over_ranks(ms, tokens, device, world):
    """Replicas exchange nothing on the data path; only the report is combined: the job's time is the
    slowest rank's, its tokens the sum over ranks.  Works on any backend (nccl on GPUs, gloo on CPU)."""
    import torch
    t_ms = torch.tensor([ms], dtype=torch.float64, device=device)
    tok = torch.tensor([tokens], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t_ms, op=dist.ReduceOp.MAX)
        dist.all_reduce(tok, op=dist.ReduceOp.SUM)
    return float(t_ms.item()), float(tok.item())


def percentiles(x):
    if len(x) == 0:
        return dict(p50=None, p99=None, mean=None)
    return dict(p50=float(np.percentile(x, 50)), p99=float(np.percentile(x, 99)), mean=float(np.mean(x)))


def realtime_run(B, m, sched, wbuf, kv, reqs, time_limit_s, use_arrivals=True, weights_layout=0, exec_mode=None):
    """Persistent loop (or, for the comparison arm, the host-driven loop of the same kernels), requests
    submitted at their arrival times from host buffers, tokens read back with blink_poll.  Returns
    throughput and latency figures."""
    eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_PERSISTENT if exec_mode is None else exec_mode,
                  stats_iters=1 << 17, idle_exit_us=2_000_000,
                  weights_layout=weights_layout, policy=POLICY)
    try:
        off = eng.blink_get_stats().device_clock_offset_ns
        n_expected = 0
        evs = []
        t0 = time.monotonic()
        t0_ns = time.monotonic_ns()
        i = 0
        got = 0
        done_req = 0
        while True:
            now = time.monotonic() - t0
            while i < len(reqs) and (not use_arrivals or reqs[i].arrival_s <= now):
                rc = eng.submit_request(reqs[i], raise_on_error=False)
                if rc == B.BLINK_EAGAIN:
                    break
                if rc < 0:
                    raise B.BlinkError(rc, "blink_submit")
                n_expected += reqs[i].max_new
                i += 1
            e = eng.blink_poll(4096, 200)
            if len(e):
                evs.append(e)
                got += len(e)
                done_req += int(e["is_last"].sum())
            if (i == len(reqs) and got >= n_expected) or now > time_limit_s:
                break
        elapsed = time.monotonic() - t0
        st = eng.blink_get_stats()
        ev = np.concatenate(evs) if evs else np.zeros(0, dtype=B.EVENT_DTYPE)
        its = int(st.iterations)
        # device-side figures (token publish times on the device clock): the paper's claim, its frontend
        # sits on the SmartNIC and not on the interfered host; host-side figures (when blink_poll saw
        # the token) and the submit lag show what the stand-in frontend on the host adds
        ttft, tpot, ttft_h, tpot_h, lag = [], [], [], [], []
        done_s = {}   # ticket -> seconds from the start of the run until the host saw its last token
        by_ticket = {r.ticket: r for r in reqs}
        if len(ev):
            ev = np.sort(ev, order=["ticket", "index"])
            bounds = np.flatnonzero(np.diff(ev["ticket"].astype(np.int64)) != 0) + 1
            for seg in np.split(ev, bounds):
                first = seg[seg["index"] == 0]
                if len(first):
                    ttft.append((int(first["t_device_ns"][0]) + off - int(first["t_submit_ns"][0])) / 1e6)
                    ttft_h.append((int(first["t_host_ns"][0]) - int(first["t_submit_ns"][0])) / 1e6)
                    if use_arrivals:
                        arr_ns = t0_ns + int(by_ticket[int(first["ticket"][0])].arrival_s * 1e9)
                        lag.append((int(first["t_submit_ns"][0]) - arr_ns) / 1e6)
                if seg["is_last"][-1]:
                    done_s[int(seg["ticket"][-1])] = (int(seg["t_host_ns"][-1]) - t0_ns) / 1e9
                if seg["is_last"][-1] and len(seg) > 1:
                    tpot.append((int(seg["t_device_ns"][-1]) - int(seg["t_device_ns"][0])) / 1e6 / (len(seg) - 1))
                    tpot_h.append((int(seg["t_host_ns"][-1]) - int(seg["t_host_ns"][0])) / 1e6 / (len(seg) - 1))
        return dict(tokens=got, elapsed_s=elapsed, tok_s=got / elapsed if elapsed > 0 else 0.0,
                    requests_submitted=i, requests_completed=done_req, iterations=its,
                    h2d_bytes=int(st.bytes_to_device), d2h_bytes=int(st.bytes_from_device),
                    ttft_ms=percentiles(ttft), tpot_ms=percentiles(tpot),
                    ttft_host_ms=percentiles(ttft_h), tpot_host_ms=percentiles(tpot_h), submit_lag_ms=percentiles(lag),
                    done_s=done_s, device_status=int(st.device_status))
    finally:
        rc = eng.blink_destroy()
        if rc != B.BLINK_OK:
            log(f"blink_destroy returned {rc}")


# ----------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="blink", choices=["blink", "reference"])
    ap.add_argument("--host-driven", default="graph", choices=["off", "graph", "launches"],
                    help="also run the latency legs with the host-driven loop of the same kernels (comparison arm)")
    ap.add_argument("--config", type=int, default=3, help="BASELINE configuration (1..5)")
    ap.add_argument("--ramp", type=int, default=-1, help="untimed iterations that bring the batch to steady state")
    ap.add_argument("--gemm", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--weights", default="streaming", choices=["streaming", "row-major"],
                    help="storage of the GEMM matrices: tile-contiguous streaming layout or plain row-major")
    ap.add_argument("--rate", type=float, default=16.0, help="offered load of the real-time run (req/s)")
    ap.add_argument("--e2e-seconds", type=float, default=15.0)
    ap.add_argument("--latency-seconds", type=float, default=20.0)
    ap.add_argument("--interfere", default="both", choices=["both", "off", "on"],
                    help="real-time run with the host idle, with the host-CPU stressor, or both (default: both, with ratios)")
    ap.add_argument("--rates", default="", help="offered-load sweep, e.g. 'all' (the 13 levels) or '4,8,16': one real-time run per "
                    "rate; reports the highest rate whose goodput reaches 0.95 x offered")
    ap.add_argument("--rate-seconds", type=float, default=30.0, help="measurement window per rate of the sweep")
    ap.add_argument("--skip-parity", action="store_true")
    ap.add_argument("--print-digest", action="store_true", help="print kernel_digest() and exit")
    ap.add_argument("--policy", default="chunked", choices=["chunked", "pause-resume"],
                    help="chunked prefill (default), or the paper's whole-prompt prefill steps that pause decoding")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-latency", action="store_true")
    ap.add_argument("--closed-batch", default="", help="N,I,O: use an N x I -> O closed batch instead of the stream")
    ap.add_argument("--kv-fraction", type=float, default=0.8)
    ap.add_argument("--kv-blocks", type=int, default=0, help="cap the KV pool at this many blocks")
    ap.add_argument("--decode-points", default="64,512,256;256,512,384",
                    help="N,I,O closed batches whose decode steps are timed besides the stream ('' = none)")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: keep only this many layers of the configuration's shape")
    ap.add_argument("--exec", default="manual", choices=["manual", "stepped"],
                    help="stepped = one host launch per phase (profiling aid for ncu; prints no bench value)")
    args = ap.parse_args()

    if args.print_digest:
        print(kernel_digest())
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    from synth import make_requests, model_cfg, sched_cfg
    from synth.workload import closed_batch
    cfg_i = args.config
    m = model_cfg(cfg_i)
    if args.layers > 0:
        m = m.with_(n_layers=args.layers)
    sched = sched_cfg(cfg_i)
    if args.policy == "pause-resume":
        global POLICY
        POLICY = 1
        sched = sched.with_(prefill_chunk_tokens=max(sched.prefill_chunk_tokens, sched.max_prompt))
    workload = f"C{cfg_i} {('8B' if cfg_i in (3, 4) else '')} stream".replace("  ", " ")
    if args.layers > 0:
        workload += f" ({args.layers} layers only)"

    if args.impl == "reference":
        if rank != 0:
            return
        import torch
        from synth import make_weights
        dev = "cuda:0" if torch.cuda.is_available() and cfg_i >= 3 else "cpu"
        if cfg_i == 5:   # the 93 GB model does not fit the host in fp32: two layers of the same shape
            m = m.with_(n_layers=2)
            workload += " (two-layer model of the same layer shape)"
        wbuf = make_weights(m, 20260407, dev)
        n_req, cap, new = (4, 64, 8) if cfg_i >= 2 else (8, 64, 32)
        vals = []
        for _ in range(max(1, min(args.steps, 3))):
            cb, res, dt = cpu_oracle_sample(m, sched, wbuf, n_req, cap, new, cfg_i)
            vals.append(cb["value"])
        cb["value"] = float(np.median(vals))
        line = dict(impl="reference", metric="output tok/s", value=cb["value"], unit="tok/s", n_gpus=args.gpus,
                    steps=args.steps, warmup=args.warmup, ms_per_step=dt * 1e3 / max(1, len(res["trace"])),
                    higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32", data="synthetic",
                    config=dict(workload=workload + " (bounded sample, CPU oracle)"), cpu_baseline=cb,
                    e2e=dict(value=cb["value"], unit="tok/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
        print(json.dumps(line), flush=True)
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the serving loop has no CPU fallback")
    from paper_2604_07609_b200 import binding as B
    from paper_2604_07609_b200 import build as Bbuild
    from synth import make_weights
    Bbuild.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device(f"cuda:{local_rank}")
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    gemm_impl = dict(auto=B.GEMM_AUTO, simt=B.GEMM_SIMT, tc=B.GEMM_TC)[args.gemm]
    t_setup = time.time()
    wbuf = make_weights(m, 20260407 + rank, dev)
    torch.cuda.synchronize()
    log(f"[bench] weights {wbuf.numel() / 1e9:.2f} GB on {dev} in {time.time() - t_setup:.1f}s")

    # ---- CPU oracle beside it (rank 0, N = 1 only) ----------------------------------------
    cpu_baseline, cpu_res = None, None
    if rank == 0 and world == 1 and not args.skip_cpu:
        try:
            n_req, cap, new = (4, 64, 8) if cfg_i >= 2 else (8, 64, 32)
            if cfg_i == 5:
                # the routed-expert model (93 GB in bf16) does not fit the host in fp32: the oracle is timed on a
                # two-layer model of the same layer shape with weights of its own
                m2 = m.with_(n_layers=2)
                cpu_baseline, cpu_res, _ = cpu_oracle_sample(m2, sched, make_weights(m2, 20260407, "cpu"), n_req, cap, new, cfg_i)
                cpu_baseline["sample"] = "TWO-LAYER model of the same layer shape (the full model does not fit the host): " + \
                    cpu_baseline["sample"]
            else:
                cpu_baseline, cpu_res, _ = cpu_oracle_sample(m, sched, wbuf, n_req, cap, new, cfg_i,
                                                             keep_logits=not args.skip_parity)
            log(f"[bench] cpu oracle: {cpu_baseline['value']:.2f} tok/s ({cpu_baseline['sample']})")
        except Exception as e:  # a baseline, never a reason to lose the measurement
            cpu_baseline = dict(value=None, unit="output tok/s", cores=os.cpu_count(), kind="oracle",
                                sample=f"failed: {e!r}")

    wl = B.WEIGHTS_ROW_MAJOR
    if args.weights == "streaming" and m.dtype == "bf16" and args.gemm != "simt":
        B.blink_convert_weights(m, wbuf, B.WEIGHTS_ROW_MAJOR, B.WEIGHTS_STREAMING)   # set-up, once, in place
        wl = B.WEIGHTS_STREAMING
    parity = None
    if cpu_res is not None and "plain" in cpu_res:
        try:
            parity = parity_on_sample(B, m, wbuf, wl, cpu_res)
            log(f"[bench] parity on the oracle sample: max-abs {parity['parity_max_abs']:.3e} (the two oracles differ by "
                f"{parity['oracle_rounding_noise_max_abs']:.3e}), trace equal: {parity['trace_equal']}")
        except Exception as e:
            parity = dict(parity_max_abs=None, note=f"failed: {e!r}")
        cpu_res = None
    # ---- KV pool: a fraction of what is free after the weights ---------------------------
    free, total = torch.cuda.mem_get_info(dev)
    lib_reserve = 6 << 30      # ring, arenas, activations and logits the library allocates itself
    blk = B.kv_bytes_per_block(m, sched.block_size)
    n_blocks = int((free - lib_reserve) * args.kv_fraction) // blk
    if sched.n_blocks > 0:
        n_blocks = min(n_blocks, sched.n_blocks)
    if args.kv_blocks > 0:
        n_blocks = min(n_blocks, args.kv_blocks)
    kv = torch.empty(n_blocks * blk, dtype=torch.uint8, device=dev)
    sched = sched.with_(n_blocks=n_blocks)
    log(f"[bench] KV pool {n_blocks} blocks = {n_blocks * blk / 1e9:.1f} GB ({n_blocks * 16} tokens)")

    if args.closed_batch:
        n, i_len, o_len = (int(x) for x in args.closed_batch.split(","))
        reqs = closed_batch(n, i_len, o_len, m.vocab, seed=7, top_k=50 if cfg_i >= 3 else 0, temperature=0.8)
        workload = f"C{cfg_i} shape, closed batch {n}x{i_len}->{o_len}"
        ramp = args.ramp if args.ramp >= 0 else (n * i_len + sched.prefill_chunk_tokens - 1) // sched.prefill_chunk_tokens + 2
    else:
        reqs = make_requests(cfg_i, rate=args.rate)
        # untimed iterations that bring the batch to its steady composition (the short streams of the small
        # configurations drain earlier)
        ramp = args.ramp if args.ramp >= 0 else {1: 4, 2: 150, 5: 300}.get(cfg_i, 600)

    W, K = max(3, args.warmup), args.steps
    if args.exec == "stepped":
        # profiling aid: the same device code, one host launch per phase, so that a profiler sees
        # the phases as separate kernels (1 control launch + 9 per layer + 3 per iteration)
        eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_STEPPED, gemm_impl=gemm_impl, stats_iters=ramp + W + K + 64,
                      weights_layout=wl, policy=POLICY)
        try:
            for r in reqs:
                eng.submit_request(r)
            eng.blink_step(ramp + W)
            eng.blink_poll(4096, 0)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            eng.blink_step(K)
            dt = time.perf_counter() - t0
            its = eng.blink_get_iter_stats()[-K:]
            by_s, _ = step_bytes_flops(m, its)
            by_full, _ = step_bytes_flops(model_cfg(cfg_i), its)
            print(json.dumps(dict(mode="stepped (profiling aid, not a bench value)", workload=workload, steps=K,
                                  algorithmic_gb_per_step=float(by_s.mean() / 1e9),
                                  algorithmic_gb_per_step_full_layer_count=float(by_full.mean() / 1e9),
                                  kv_tokens_per_step=float(its["kv_tokens"].mean()), kernel_digest=kernel_digest(),
                                  wall_ms_per_step=dt * 1e3 / K, rows_per_step=float(its["n_tokens"].mean()),
                                  decode_rows_per_step=float(its["n_decode"].mean()),
                                  launches_per_step=1 + 9 * m.n_layers + 3)), flush=True)
        finally:
            eng.blink_destroy()
        return

    # ---- closed-loop saturation run: ramp, W warm-up steps, then exactly K timed steps --------
    eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_MANUAL, gemm_impl=gemm_impl, stats_iters=ramp + W + K + 64,
                  idle_exit_us=200_000, weights_layout=wl, policy=POLICY)
    try:
        for r in reqs:
            eng.submit_request(r)
        t0 = time.time()
        if ramp > 0:
            ramp_ms = eng.blink_run(ramp)
            eng.blink_poll(4096, 0)
            log(f"[bench] ramp {ramp} iterations in {ramp_ms / 1e3:.1f}s")
        eng.blink_run(W)
        while len(eng.blink_poll(4096, 0)):
            pass
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        clocks = ClockSampler(local_rank)
        clocks.start()
        it0 = int(eng.blink_get_stats().iterations)
        ms = eng.blink_run(K)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        clk = clocks.stop()
        st = eng.blink_get_stats()
        its = eng.blink_get_iter_stats()[it0:it0 + K]
        done_iters = int(st.iterations) - it0
        if st.device_status not in (0,):
            raise SystemExit(f"device status {st.device_status}")
        if done_iters != K:
            raise SystemExit(f"the workload ran dry after {done_iters} of {K} timed steps: lower --ramp/--steps")
    finally:
        eng.blink_destroy()

    tokens_out = int(its["n_sample_rows"].sum())
    by, fl = step_bytes_flops(m, its)
    pk = measured_peaks()
    ms_max, tok_all = reduce_over_ranks(ms, tokens_out, dev, world)
    value = tok_all / (ms_max / 1e3)

    bound_hbm_s = by / (pk["hbm_gbs"] * 1e9)
    bound_tc_s = fl / (pk["tf_sustained"] * 1e12)
    hbm_bound = bound_hbm_s.sum() >= bound_tc_s.sum()
    if hbm_bound:
        roof = dict(bound="hbm", achieved=float(by.sum() / (ms / 1e3) / 1e9), peak=pk["hbm_gbs"], unit="GB/s")
    else:
        roof = dict(bound="tensor", achieved=float(fl.sum() / (ms / 1e3) / 1e12), peak=pk["tf_sustained"],
                    unit="TFLOP/s")
    roof["frac"] = roof["achieved"] / roof["peak"]
    tr = TRAFFIC.get(workload)
    if tr and tr["digest"] == kernel_digest() and tr["algorithmic_gb"] > 0:
        # bytes per launch (one launch = the K timed steps), like `achieved`
        roof["traffic"] = float(tr["traffic_gb"] * 1e9 * (by.sum() / 1e9) / tr["algorithmic_gb"])
        roof["traffic_over_algorithmic"] = tr["traffic_gb"] / tr["algorithmic_gb"]
        roof["traffic_source"] = tr["source"]
    else:
        roof["traffic"] = None   # no capture for this workload, or the kernels changed since it was taken
    roof["peak_source"] = pk["source"]
    roof["kernel"] = "blink_loop_kernel (one launch = the K timed steps)"
    roof["algorithmic_gb_per_step"] = float(by.mean() / 1e9)
    roof["algorithmic_tflop_per_step"] = float(fl.mean() / 1e12)
    roof["frac_of_max_bound"] = float(np.maximum(bound_hbm_s, bound_tc_s).sum() / (ms / 1e3))
    roof["frac_of_8TBs_spec"] = float(by.sum() / (ms / 1e3) / 8e12)
    step_dev_ms = (its["t_end_ns"].astype(np.int64) - its["t_begin_ns"].astype(np.int64)) / 1e6
    ctrl_us = (its["t_forward_ns"].astype(np.int64) - its["t_begin_ns"].astype(np.int64)) / 1e3

    line = dict(metric="output tok/s", value=value, unit="tok/s", n_gpus=world, steps=K, warmup=W,
                ms_per_step=ms_max / K, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16" if m.dtype == "bf16" else "f32", data="synthetic",
                config=dict(workload=workload, requests=len(reqs), max_batch=sched.max_batch,
                            prefill_chunk_tokens=sched.prefill_chunk_tokens, kv_blocks=n_blocks,
                            ramp_iterations=ramp, sampling="top-k 50, T 0.8" if cfg_i in (3, 4) else "greedy",
                            l2="per-step inputs (weights + KV) exceed L2 many times over; no flush needed",
                            rows_per_step=float(its["n_tokens"].mean()),
                            decode_rows_per_step=float(its["n_decode"].mean()),
                            parallelism="replicas" if world > 1 else "1 GPU", gemm=args.gemm, policy=args.policy,
                            weights_layout="streaming" if wl else "row-major"),
                gpu_launches=1, clocks=clk, roofline=roof,
                step_ms_device=dict(p50=float(np.median(step_dev_ms)), max=float(step_dev_ms.max())),
                phase_ms_per_step={n: float(its["phase_ns"][:, i].mean() / 1e6) for i, n in enumerate(B.PHASE_NAMES)},
                control_plane_us=dict(p50=float(np.median(ctrl_us)), max=float(ctrl_us.max())))
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    if parity is not None:
        line["parity"] = parity

    # ---- decode-only operating points (fixed batch): the HBM-bound regime ---------------------
    if args.decode_points and rank == 0 and world == 1 and not args.closed_batch:
        pts = []
        for spec in args.decode_points.split(";"):
            n, i_len, o_len = (int(v) for v in spec.split(","))
            pts.append(decode_point(B, m, sched, wbuf, kv, wl, gemm_impl, n, i_len, o_len, 20, cfg_i))
            log(f"[bench] decode point {spec}: {pts[-1]['ms_per_step']:.2f} ms/step, "
                f"{pts[-1]['frac_of_measured_hbm']:.3f} of measured HBM")
        line["decode_steps"] = pts

    # ---- end to end through the public API with host buffers ------------------------------
    if not args.skip_e2e:
        r = realtime_run(B, m, sched, wbuf, kv, reqs, args.e2e_seconds, use_arrivals=False, weights_layout=wl)
        e_val = torch.tensor([r["tok_s"]], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(e_val, op=dist.ReduceOp.SUM)
        itn = max(1, r["iterations"])
        line["e2e"] = dict(value=float(e_val.item()), unit="tok/s", h2d_bytes_per_step=r["h2d_bytes"] / itn,
                           d2h_bytes_per_step=r["d2h_bytes"] / itn, seconds=r["elapsed_s"], tokens=r["tokens"],
                           requests_completed=r["requests_completed"], iterations=r["iterations"],
                           note="all requests submitted from host memory at t=0 through blink_submit, tokens "
                                "read with blink_poll, persistent loop; wall clock from first submit")
    # ---- real-time run at the offered load: latency, host idle and host stressed -----------------
    def latency_leg(stressed, rate_reqs, seconds, exec_mode=None):
        stress = Stressor() if stressed else None
        if stress:
            stress.start()
        try:
            lreqs = [q for q in rate_reqs if q.arrival_s <= seconds]
            r = realtime_run(B, m, sched, wbuf, kv, lreqs, seconds * 3, use_arrivals=True, weights_layout=wl,
                             exec_mode=exec_mode)
        finally:
            if stress:
                stress.stop()
        offered_tok = sum(q.max_new for q in lreqs)
        return dict(host="stressed" if stressed else "idle", requests=len(lreqs), completed=r["requests_completed"],
                    tok_s=r["tok_s"], goodput_req_s=r["requests_completed"] / r["elapsed_s"] if r["elapsed_s"] > 0 else 0.0,
                    tokens=r["tokens"], offered_tokens=offered_tok, ttft_ms=r["ttft_ms"], tpot_ms=r["tpot_ms"],
                    ttft_host_ms=r["ttft_host_ms"], tpot_host_ms=r["tpot_host_ms"], submit_lag_ms=r["submit_lag_ms"],
                    seconds=r["elapsed_s"], done_s=r["done_s"])

    if not args.skip_latency and rank == 0 and world == 1:
        legs = {}
        if args.interfere in ("both", "off"):
            legs["isolated"] = latency_leg(False, reqs, args.latency_seconds)
        if args.interfere in ("both", "on"):
            legs["interfered"] = latency_leg(True, reqs, args.latency_seconds)
        for v in legs.values():
            v.pop("done_s", None)
        lat = dict(offered_req_s=args.rate, **legs,
                   note="ttft_ms / tpot_ms use the device publish times (the paper's frontend sits on the SmartNIC, not on "
                        "the interfered host); *_host_ms use the time blink_poll saw the token on the (stressed) host; "
                        "submit_lag_ms = blink_submit time minus scheduled arrival")
        if "isolated" in legs and "interfered" in legs:
            a, b = legs["isolated"], legs["interfered"]
            ratio = lambda x, y: (y / x) if (x and y) else None
            # interfered / isolated, the bracketed figures of the paper's Table 7
            lat["ratios"] = dict(ttft_p99=ratio(a["ttft_ms"]["p99"], b["ttft_ms"]["p99"]),
                                 tpot_p99=ratio(a["tpot_ms"]["p99"], b["tpot_ms"]["p99"]),
                                 tpot_p50=ratio(a["tpot_ms"]["p50"], b["tpot_ms"]["p50"]),
                                 throughput=ratio(a["tok_s"], b["tok_s"]),
                                 ttft_host_p99=ratio(a["ttft_host_ms"]["p99"], b["ttft_host_ms"]["p99"]),
                                 tpot_host_p99=ratio(a["tpot_host_ms"]["p99"], b["tpot_host_ms"]["p99"]))
        line["latency"] = lat
        # ---- the same kernels driven from the host, idle and stressed (Section 6.3: what interference does to a
        # host-resident serving loop; the GPU-resident loop above is the other arm) ----
        if args.host_driven != "off":
            hmode = B.EXEC_HOST_GRAPH if args.host_driven == "graph" else B.EXEC_HOST_LAUNCHES
            hl = {}
            if args.interfere in ("both", "off"):
                hl["isolated"] = latency_leg(False, reqs, args.latency_seconds, exec_mode=hmode)
            if args.interfere in ("both", "on"):
                hl["interfered"] = latency_leg(True, reqs, args.latency_seconds, exec_mode=hmode)
            for v in hl.values():
                v.pop("done_s", None)
            hd = dict(driver="a host thread launches one iteration at a time (" +
                             ("one pre-captured CUDA graph" if args.host_driven == "graph" else "one kernel launch per phase") +
                             ") and waits for it; same device code, same requests, same offered load", **hl)
            if "isolated" in hl and "interfered" in hl:
                a, b = hl["isolated"], hl["interfered"]
                ratio = lambda x, y: (y / x) if (x and y) else None
                hd["ratios"] = dict(ttft_p99=ratio(a["ttft_ms"]["p99"], b["ttft_ms"]["p99"]),
                                    tpot_p99=ratio(a["tpot_ms"]["p99"], b["tpot_ms"]["p99"]),
                                    tpot_p50=ratio(a["tpot_ms"]["p50"], b["tpot_ms"]["p50"]),
                                    throughput=ratio(a["tok_s"], b["tok_s"]))
            if not args.skip_e2e:
                # closed loop (all requests at t = 0), the same run as `e2e`, for the throughput cost of the host in the loop
                rh = realtime_run(B, m, sched, wbuf, kv, reqs, args.e2e_seconds, use_arrivals=False, weights_layout=wl,
                                  exec_mode=hmode)
                hd["e2e_tok_s"] = rh["tok_s"]
                hd["e2e_tok_s_gpu_resident"] = line.get("e2e", {}).get("value")
            line["host_driven"] = hd
    # ---- offered-load sweep (Section 6.1: 13 levels between 1 and 32 req/s; Appendix C: serviceable load) ----
    if args.rates and rank == 0 and world == 1:
        from synth.workload import RATE_LEVELS
        levels = RATE_LEVELS if args.rates == "all" else [float(v) for v in args.rates.split(",")]
        sweep, serviceable = [], None
        for lv in levels:
            rr = make_requests(cfg_i, rate=float(lv))
            leg = latency_leg(False, rr, args.rate_seconds)
            leg["offered_req_s"] = float(lv)
            # window [0, W]: requests arriving in the first part of it, [0, W - D], are the offered load; those of
            # them whose last token the host saw by W are the goodput (D = 12 s or 0.4 W lets all but the very
            # longest generations finish when nothing queues)
            Wn = args.rate_seconds
            D = min(12.0, 0.4 * Wn)
            early = [q for q in rr if q.arrival_s <= Wn - D]
            good = sum(1 for q in early if leg["done_s"].get(q.ticket, 1e30) <= Wn)
            offered = len(early) / (Wn - D)
            leg["goodput_req_s"] = good / (Wn - D)
            leg["goodput_over_offered"] = good / len(early) if early else None
            leg.pop("done_s", None)
            sweep.append(leg)
            if leg["goodput_over_offered"] is not None and leg["goodput_over_offered"] >= 0.95:
                serviceable = float(lv)
            log(f"[bench] rate {lv}: goodput {leg['goodput_req_s']:.2f} req/s of {offered:.2f} offered, "
                f"TPOT p99 {leg['tpot_ms']['p99']}")
        line["rate_sweep"] = dict(levels=sweep, serviceable_req_s=serviceable,
                                  rule="highest offered rate at which at least 0.95 of the requests that arrived in the "
                                       "first W - D seconds of the W-second window had their last token by its end")
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
