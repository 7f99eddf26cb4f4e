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


def cpu_oracle_sample(m, sched, wbuf, n_requests, prompt_cap, new_tokens, config):
    """Time the oracle, as it stands, on a bounded sample of the workload."""
    import torch
    from oracle import serve as OS
    from oracle import transformer as O2
    from synth import make_requests
    reqs = make_requests(config, n_requests=n_requests)
    for r in reqs:
        r.prompt = r.prompt[:prompt_cap]
        r.max_new = new_tokens
    arrays = weights_to_host_fp32(m, wbuf)
    W = O2.Weights(m, arrays, dtype=np.float32)
    sch = sched.with_(n_blocks=max(64, n_requests * ((prompt_cap + new_tokens) // 16 + 2)))
    t0 = time.perf_counter()
    res = OS.run(m, sch, W, reqs, act_round=O2.round_bf16 if m.dtype == "bf16" else None, keep_logits=False)
    dt = time.perf_counter() - t0
    n_out = sum(len(v) for v in res["tokens"].values())
    return dict(value=n_out / dt, unit="output tok/s", cores=torch.get_num_threads(), kind="oracle",
                sample=f"first {n_requests} requests of the stream, prompts cut to {prompt_cap} tokens, "
                       f"{new_tokens} new tokens each, full {m.n_layers}-layer model in fp32 numpy; "
                       f"{n_out} tokens in {dt:.1f} s, {len(res['trace'])} iterations"), res, dt


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
                  idle_exit_us=200_000, weights_layout=wl)
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


def realtime_run(B, m, sched, wbuf, kv, reqs, time_limit_s, use_arrivals=True, weights_layout=0):
    """Persistent loop, requests submitted at their arrival times from host buffers, tokens
    read back with blink_poll.  Returns throughput and latency figures."""
    eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_PERSISTENT, stats_iters=1 << 17, idle_exit_us=2_000_000,
                  weights_layout=weights_layout)
    try:
        off = eng.blink_get_stats().device_clock_offset_ns
        n_expected = 0
        evs = []
        t0 = time.monotonic()
        i = 0
        h2d = 0
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
                h2d += reqs[i].n_prompt * 4 + 64
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
        ttft, tpot = [], []
        if len(ev):
            ev = np.sort(ev, order=["ticket", "index"])
            bounds = np.flatnonzero(np.diff(ev["ticket"].astype(np.int64)) != 0) + 1
            for seg in np.split(ev, bounds):
                first = seg[seg["index"] == 0]
                if len(first):
                    ttft.append((int(first["t_device_ns"][0]) + off - int(first["t_submit_ns"][0])) / 1e6)
                if seg["is_last"][-1] and len(seg) > 1:
                    tpot.append((int(seg["t_device_ns"][-1]) - int(seg["t_device_ns"][0])) / 1e6 / (len(seg) - 1))
        return dict(tokens=got, elapsed_s=elapsed, tok_s=got / elapsed if elapsed > 0 else 0.0,
                    requests_submitted=i, requests_completed=done_req, iterations=its,
                    h2d_bytes=h2d, d2h_bytes=got * 16, ttft_ms=percentiles(ttft), tpot_ms=percentiles(tpot),
                    device_status=int(st.device_status))
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
    ap.add_argument("--config", type=int, default=3, help="BASELINE configuration (1..4)")
    ap.add_argument("--ramp", type=int, default=-1, help="untimed iterations that bring the batch to steady state")
    ap.add_argument("--gemm", default="auto", choices=["auto", "simt", "tc"])
    ap.add_argument("--weights", default="streaming", choices=["streaming", "row-major"],
                    help="storage of the GEMM matrices: tile-contiguous streaming layout or plain row-major")
    ap.add_argument("--rate", type=float, default=16.0, help="offered load of the real-time run (req/s)")
    ap.add_argument("--e2e-seconds", type=float, default=15.0)
    ap.add_argument("--latency-seconds", type=float, default=20.0)
    ap.add_argument("--interfere", action="store_true", help="run the host-CPU stressor during the real-time run")
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
    workload = f"C{cfg_i} {('8B' if cfg_i in (3, 4) else '')} stream".replace("  ", " ")
    if args.layers > 0:
        workload += f" ({args.layers} layers only)"

    if args.impl == "reference":
        if rank != 0:
            return
        import torch
        from synth import make_weights
        dev = "cuda:0" if torch.cuda.is_available() and cfg_i >= 3 else "cpu"
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
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        try:
            n_req, cap, new = (4, 64, 8) if cfg_i >= 2 else (8, 64, 32)
            cpu_baseline, _, _ = cpu_oracle_sample(m, sched, wbuf, n_req, cap, new, cfg_i)
            log(f"[bench] cpu oracle: {cpu_baseline['value']:.2f} tok/s ({cpu_baseline['sample']})")
        except Exception as e:  # a baseline, never a reason to lose the measurement
            cpu_baseline = dict(value=None, unit="output tok/s", cores=os.cpu_count(), kind="oracle",
                                sample=f"failed: {e!r}")

    wl = B.WEIGHTS_ROW_MAJOR
    if args.weights == "streaming" and m.dtype == "bf16" and args.gemm != "simt":
        B.blink_convert_weights(m, wbuf, B.WEIGHTS_ROW_MAJOR, B.WEIGHTS_STREAMING)   # set-up, once, in place
        wl = B.WEIGHTS_STREAMING
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
        ramp = args.ramp if args.ramp >= 0 else 600

    W, K = max(3, args.warmup), args.steps
    if args.exec == "stepped":
        # profiling aid: the same device code, one host launch per phase, so that a profiler sees
        # the phases as separate kernels (1 control launch + 9 per layer + 3 per iteration)
        eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_STEPPED, gemm_impl=gemm_impl, stats_iters=ramp + W + K + 64,
                      weights_layout=wl)
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
            print(json.dumps(dict(mode="stepped (profiling aid, not a bench value)", workload=workload, steps=K,
                                  wall_ms_per_step=dt * 1e3 / K, rows_per_step=float(its["n_tokens"].mean()),
                                  decode_rows_per_step=float(its["n_decode"].mean()),
                                  launches_per_step=1 + 9 * m.n_layers + 3)), flush=True)
        finally:
            eng.blink_destroy()
        return

    # ---- closed-loop saturation run: ramp, W warm-up steps, then exactly K timed steps --------
    eng = B.Blink(m, sched, wbuf, kv, exec_mode=B.EXEC_MANUAL, gemm_impl=gemm_impl, stats_iters=ramp + W + K + 64,
                  idle_exit_us=200_000, weights_layout=wl)
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
    roof["traffic"] = None
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
                            ramp_iterations=ramp, sampling="top-k 50, T 0.8" if cfg_i >= 3 else "greedy",
                            l2="per-step inputs (weights + KV) exceed L2 many times over; no flush needed",
                            rows_per_step=float(its["n_tokens"].mean()),
                            decode_rows_per_step=float(its["n_decode"].mean()),
                            parallelism="replicas" if world > 1 else "1 GPU", gemm=args.gemm,
                            weights_layout="streaming" if wl else "row-major"),
                gpu_launches=1, clocks=clk, roofline=roof,
                step_ms_device=dict(p50=float(np.median(step_dev_ms)), max=float(step_dev_ms.max())),
                phase_ms_per_step={n: float(its["phase_ns"][:, i].mean() / 1e6) for i, n in enumerate(B.PHASE_NAMES)},
                control_plane_us=dict(p50=float(np.median(ctrl_us)), max=float(ctrl_us.max())))
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline

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
    # ---- real-time run at the offered load: latency ----------------------------------------
    if not args.skip_latency and rank == 0 and world == 1:
        stress = Stressor() if args.interfere else None
        if stress:
            stress.start()
        try:
            lreqs = [q for q in reqs if q.arrival_s <= args.latency_seconds]
            r = realtime_run(B, m, sched, wbuf, kv, lreqs, args.latency_seconds * 3, use_arrivals=True, weights_layout=wl)
        finally:
            if stress:
                stress.stop()
        line["latency"] = dict(offered_req_s=args.rate, host="stressed" if args.interfere else "idle",
                               requests=len(lreqs), completed=r["requests_completed"], tok_s=r["tok_s"],
                               ttft_ms=r["ttft_ms"], tpot_ms=r["tpot_ms"], seconds=r["elapsed_s"])
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
