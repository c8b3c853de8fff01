"""Benchmark of the SSD verify step (one pass of the whole hot path = one "step").

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config C]

Workload at N = 1: the Qwen2-style target (24 layers, hidden 896), batch 1, gamma = 4, prefix 300,
bf16 weights and KV cache (configs[1]); inputs are seeded and synthetic.  A step runs
ssd_verify + ssd_kv_commit + ssd_kv_restore (the restore puts the stream back on the same prefix
so every step does identical work) as one CUDA-graph launch on data already resident in HBM;
`e2e` runs the host-buffer entry point with its H2D / D2H copies inside the timed region.
For N > 1 each rank runs an independent replica (streams are independent; no collective).

Prints ONE JSON line.  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

NOMINAL_HBM_GBS = 8000.0
KERNEL_SOURCES = ("fast_kernel.cuh", "fast.h", "fast_verify.cu", "fast_pack.cu")


def kernel_sources_sha1():
    """Hash of the persistent forward kernel's sources: ties a profile summary to the code it measured."""
    import hashlib
    h = hashlib.sha1()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2505_15380_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def profiled_traffic(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the persistent forward kernel,
    read from the ncu summary under profiles/; None when there is no summary for this workload or
    the kernel's sources have changed since it was taken."""
    path = os.path.join(ROOT, "profiles", f"fast_forward_kernel_{workload}_ncu_sections.md")
    if not os.path.exists(path):
        return None
    fields = {}
    for line in open(path):
        if ":" in line:
            k, v = line.split(":", 1)
            fields[k.strip().strip("`*- ")] = v.strip().strip("`")
    if fields.get("kernel_sources_sha1") != kernel_sources_sha1():
        return None
    try:
        return int(fields["dram_bytes_per_launch"])
    except (KeyError, ValueError):
        return None


def _measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f).get("hbm_gbs"), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        # samples under load: the upper half of the observed clocks
        sm.sort()
        load = sm[len(sm) // 2:] if sm else []
        return {"sm_mhz": statistics.median(load) if load else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(wl, steps: int, warmup: int):
    """Times the CPU oracle's verify step (forward + transform + accept + commit) as it stands."""
    from oracle import ssd_oracle as orc
    from paper_2505_15380_b200 import synth
    shape = wl.target
    w = synth.make_weights(shape, wl.model_seed)
    m = orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                  n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn,
                  vocab_out=shape.vocab_out, vocab_text=shape.vocab_text,
                  rope_theta=shape.rope_theta, rms_eps=shape.rms_eps,
                  kv_bf16=shape.weight_dtype == synth.BF16, weights=w)
    n = wl.prefix_lens[0] - 1
    st = orc.Stream(m, n + 64)
    rng = np.random.Generator(np.random.Philox(key=99))
    for l in range(m.L):       # seeded random prefix K/V (timing only; a prefill costs the same per row)
        st.K[l][:n] = synth.bf16_round((rng.standard_normal((n, m.Hkv, m.hd)) * 0.6).astype(np.float32))
        st.V[l][:n] = synth.bf16_round((rng.standard_normal((n, m.Hkv, m.hd)) * 0.6).astype(np.float32))
    st.length, st.pending = n, 5
    V, g = shape.vocab_out, wl.gamma
    p = synth.random_prob_rows(g, V, 1)
    x = synth.sample_from_rows(p, 2)
    u = synth.verify_uniforms(0, 1, g + 1)[0]
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        r = orc.verify(m, st, x, p, u, temperature=wl.temperature, top_k=wl.top_k, beta=0.4)
        orc.commit(st, r["k"], r["y"])
        times.append(time.perf_counter() - t0)
        orc.truncate(st, n, 5)
    try:
        import threadpoolctl
        threads = max((d.get("num_threads", 1) for d in threadpoolctl.threadpool_info()), default=1)
    except Exception:
        threads = os.cpu_count() or 1
    return times[warmup:], threads


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2505_15380_b200 import synth
    wl = synth.workload(args.config)
    steps, warmup = min(args.steps, 10), min(args.warmup, 2)
    times, threads = oracle_sample(wl, steps, warmup)
    us = 1e6 * sum(times) / len(times)
    sample = (f"{len(times)} verify steps of stream 0 ({wl.gamma + 1} rows, prefix "
              f"{wl.prefix_lens[0]}, synthetic K/V), float64 numpy")
    out = {"impl": "reference", "metric": "verify_step_us", "value": us, "unit": "us",
           "n_gpus": args.gpus, "steps": len(times), "warmup": warmup, "ms_per_step": us / 1e3,
           "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic",
           "config": {"workload": wl.name, "batch": wl.batch, "gamma": wl.gamma,
                      "prefix": wl.prefix_lens[0]},
           "cpu_baseline": {"value": us, "unit": "us", "cores": threads, "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def run_loop(args, wl, tmodel, dev, beta):
    """Algorithm 1 as a whole on the device: one captured ssd_iteration (gamma draft steps of the
    workload's draft model, verify, accept, both commits, emitted tokens) replayed n times with no
    host work in between.  Returns speech tokens per second per stream and acceptance statistics."""
    import torch
    from paper_2505_15380_b200 import binding, synth
    B, g = wl.batch, wl.gamma
    n = args.loop_iterations
    dshape = wl.draft
    dmodel = binding.Model(dshape, synth.weights_blob(dshape, synth.make_weights(dshape, wl.model_seed + 500)),
                           device=dev)
    cap = max(wl.prefix_lens) + (n + 4) * (g + 1) + g + 8
    ts, ds = binding.Streams(tmodel, B, cap, g), binding.Streams(dmodel, B, cap, g)
    prefixes = [synth.make_prefix(wl, b) for b in range(B)]
    ts.prefill(prefixes)
    ds.prefill(prefixes)
    per = g + 2 * (g + 1)
    pool = np.stack([synth.verify_uniforms(wl.data_seed + 11, B, per, step=it)[:, :, 0]
                     for it in range(n + 4)]).astype(np.float32)
    loop = binding.Loop(ts, ds, prefixes, g, pool, out_capacity=(n + 4) * (g + 1))
    par = binding.VerifyParams(g, wl.temperature, wl.top_k, beta)
    L = binding.lib()
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for _ in range(3):                       # warm-up iterations (they advance the streams)
            loop.iterate(par, stream=stream)
        stream.synchronize()
        n0 = L.ssd_kernel_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            loop.iterate(par, stream=stream)
        launches = L.ssd_kernel_launch_count() - n0
        c0 = loop.out_count.clone()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
    ms = e0.elapsed_time(e1)
    assert ts.last_status() == 0 and ds.last_status() == 0
    emitted = (loop.out_count - c0).cpu().numpy().astype(np.float64)
    log = loop.accept_log.cpu().numpy()[3:3 + n]
    tested = np.minimum(log + 1, g).sum()
    alpha = float(log.sum() / tested) if tested else 0.0
    closed = (1 - alpha ** (g + 1)) / (1 - alpha) if alpha < 1 else g + 1
    return {"speech_tokens_per_s_per_stream": float(emitted.mean() / (ms * 1e-3)),
            "iterations": n, "us_per_iteration": ms * 1e3 / n, "gpu_launches_per_iteration": int(launches),
            "mean_tokens_per_iteration": float(emitted.mean() / n),
            "per_position_acceptance_alpha": alpha,
            "closed_form_tokens_per_iteration": closed,
            "draft": f"{dshape.n_layers} layers, d {dshape.d_model}, random init",
            "note": "draft x gamma + verify + accept + both commits inside the timed region; "
                    "the prefix grows by the emitted tokens as the loop runs"}


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2505_15380_b200 import binding, replicas, synth

    world, rank, local = replicas.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.workload(args.config, gamma=args.gamma, prefix=args.prefix)
    shape = wl.target
    B, g, R, V = wl.batch, wl.gamma, wl.gamma + 1, shape.vocab_out
    w = synth.make_weights(shape, wl.model_seed)
    model = binding.Model(shape, synth.weights_blob(shape, w), device=dev)
    del w
    cap = max(wl.prefix_lens) + 2 * R + 8
    gs = binding.Streams(model, B, cap, g)
    if max(wl.prefix_lens) <= 512 and not args.synthetic_kv:
        gs.prefill([synth.make_prefix(wl, b) for b in range(B)])
    else:           # long prefixes: seeded random K/V written straight into the cache
        lens = [n - 1 for n in wl.prefix_lens]
        synth.fill_synthetic_kv(gs.kv, lens, seed=wl.data_seed + 100)
        gs.kv_truncate(lens, [int(synth.make_prefix(wl, b)[-1]) for b in range(B)])
    lens0, pend0 = gs.get_state()
    d_len0 = torch.from_numpy(lens0).to(dev)
    d_pend0 = torch.from_numpy(pend0).to(dev)

    params = binding.VerifyParams(g, wl.temperature, wl.top_k, args.beta)
    d_k = torch.zeros(B, dtype=torch.int32, device=dev)
    d_y = torch.zeros(B, dtype=torch.int32, device=dev)
    d_u = torch.from_numpy(synth.verify_uniforms(wl.data_seed, B, R)).to(dev)
    # Draft rows resembling the target: p_i = softmax((target logits_i + noise) / T), x_i ~ p_i,
    # built position by position from the CUDA path's own logits (input preparation, untimed).
    d_tok = torch.zeros((B, g), dtype=torch.int32, device=dev)
    d_p = torch.full((B, g, V), 1.0 / V, dtype=torch.float32, device=dev)
    d_logits = torch.zeros((B, R, V), dtype=torch.float32, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1234 + wl.data_seed)
    for i in range(g):
        gs.verify(d_tok, d_p, d_u, params, d_k, d_y, d_logits)
        z = (d_logits[:, i, :] + args.draft_noise * torch.randn((B, V), generator=gen, device=dev)) / wl.temperature
        if 0 < wl.top_k < V:
            kth = torch.topk(z, wl.top_k, dim=-1).values[:, -1:]
            z = torch.where(z >= kth, z, torch.full_like(z, float("-inf")))
        p = torch.softmax(z, dim=-1)
        d_p[:, i, :] = p
        d_tok[:, i] = torch.multinomial(p, 1, generator=gen)[:, 0].to(torch.int32)
    torch.cuda.synchronize()

    def step():
        gs.verify(d_tok, d_p, d_u, params, d_k, d_y, None)
        gs.kv_commit(d_k, d_y)
        gs.kv_restore(d_len0, d_pend0)

    L = binding.lib()
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        step()                                   # sets kernel attributes outside the capture
        stream.synchronize()
        n0 = L.ssd_kernel_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            step()
        launches_per_step = L.ssd_kernel_launch_count() - n0
        for _ in range(max(args.warmup, 3)):
            graph.replay()
        stream.synchronize()
        replicas.barrier(world)
        torch.cuda.synchronize()
        clocks = ClockSampler(local)
        clocks.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        replicas.barrier(world)
        dev_ms = e0.elapsed_time(e1)
        k_timed = d_k.cpu().numpy().copy()
        # the dominant kernel alone: the decoder forward (one persistent kernel when the forward has
        # at most 16 rows), in a graph of its own, timed with events on the launching stream
        fgraph = torch.cuda.CUDAGraph()
        gs.forward(d_tok, g, d_logits, stream=stream)
        stream.synchronize()
        n1 = L.ssd_kernel_launch_count()
        with torch.cuda.graph(fgraph, stream=stream):
            gs.forward(d_tok, g, d_logits, stream=stream)
        fwd_launches = L.ssd_kernel_launch_count() - n1
        for _ in range(3):
            fgraph.replay()
        stream.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for _ in range(args.steps):
            fgraph.replay()
        f1.record(stream)
        stream.synchronize()
        fwd_ms = f0.elapsed_time(f1)
        # per-step distribution (each replay between its own events)
        per = []
        for _ in range(min(args.steps, 50)):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            graph.replay()
            b.record(stream)
            b.synchronize()
            per.append(a.elapsed_time(b) * 1e3)
        # ---- end to end: host buffers through ssd_verify_host, copies inside the timed region
        h_tok = d_tok.cpu().pin_memory()
        h_p = d_p.cpu().pin_memory()
        h_u = d_u.cpu().pin_memory()
        h_k = torch.zeros(B, dtype=torch.int32).pin_memory()
        h_y = torch.zeros(B, dtype=torch.int32).pin_memory()
        for _ in range(3):
            gs.verify_host(h_tok, h_p, h_u, params, h_k, h_y, stream=stream)
            gs.kv_restore(d_len0, d_pend0, stream=stream)
        stream.synchronize()
        e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2.record(stream)
        for _ in range(args.steps):
            gs.verify_host(h_tok, h_p, h_u, params, h_k, h_y, stream=stream)
            gs.kv_restore(d_len0, d_pend0, stream=stream)
        e3.record(stream)
        stream.synchronize()
        e2e_ms = e2.elapsed_time(e3)
        clk = clocks.stop()
    assert gs.last_status() == 0, "device status flags raised during the benchmark"
    assert np.array_equal(h_k.numpy(), k_timed), "host-buffer path disagrees with the device path"
    loop_stats = None
    if args.loop_iterations > 0:
        betas = (0.0, 0.1, 0.2, 0.3, 0.4) if args.beta_sweep else (0.0, args.beta)
        loop_stats = {str(beta): run_loop(args, wl, model, dev, beta) for beta in dict.fromkeys(betas + (args.beta,))}

    dev_ms, e2e_ms, fwd_ms = replicas.slowest([dev_ms, e2e_ms, fwd_ms], world, dev)   # max over ranks
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    us = dev_ms * 1e3 / args.steps
    e2e_us = e2e_ms * 1e3 / args.steps
    kv_read = sum(int(n) + R for n in lens0) * shape.kv_bytes_per_token()
    alg_bytes = shape.streamed_weight_bytes() + kv_read
    fwd_us = fwd_ms * 1e3 / args.steps
    persistent = fwd_launches == 1
    # roofline of the dominant kernel: the persistent forward kernel when there is one (it streams
    # all algorithmic bytes of the step), else the step as a whole
    kern_us = fwd_us if persistent else us
    achieved = alg_bytes / (kern_us * 1e-6) / 1e9
    peak, peak_kind = _measured_peaks()
    mean_tokens = float(np.mean(k_timed + 1))
    out = {
        "metric": "verify_step_us", "value": us, "unit": "us", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": us / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if shape.weight_dtype == synth.BF16 else "f32", "data": "synthetic",
        "config": {"workload": wl.name, "batch": B, "gamma": g, "prefix": list(wl.prefix_lens)[:4],
                   "temperature": wl.temperature, "top_k": wl.top_k, "beta": args.beta,
                   "l2": "inputs (weights %.0f MB) exceed the 126 MB L2; no flush" %
                         (shape.streamed_weight_bytes() / 1e6),
                   "replicas": world},
        "verify_step_us_p10_p50_p90": [float(np.percentile(per, q)) for q in (10, 50, 90)],
        "verify_steps_per_s_total": world * 1e6 / us,
        "speech_tokens_per_s_per_stream": (
            {"value": loop_stats[str(args.beta)]["speech_tokens_per_s_per_stream"],
             "by_beta": loop_stats,
             "note": "whole SSD iterations (Algorithm 1) run from the device, drafting included"}
            if loop_stats else
            {"value": mean_tokens * 1e6 / us, "mean_tokens_per_step": mean_tokens,
             "note": "verify-only (loop not run): drafting time not included"}),
        "e2e": {"value": e2e_us, "unit": "us",
                "h2d_bytes_per_step": B * g * 4 + B * g * V * 4 + B * R * 8,
                "d2h_bytes_per_step": B * 8},
        "gpu_launches": int(launches_per_step) * args.steps,
        "gpu_launches_per_step": int(launches_per_step),
        "clocks": clk,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_8TBps": achieved / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_step": alg_bytes, "traffic": profiled_traffic(wl.name) if persistent else None,
                     "kernel": ("fast_forward_kernel (persistent decoder forward, one launch)" if persistent
                                else "whole verify step (all launches of one graph replay)"),
                     "kernel_us": kern_us, "kernel_share_of_step": kern_us / us,
                     "step_frac": alg_bytes / (us * 1e-6) / 1e9 / peak},
        "paper_context": "paper reports 1.4x LM speedup over AR decoding on A100-SXM4-40GB "
                         "(beta=0.4, L_d=3); no verify-step latency is published",
    }
    if not args.no_cpu_baseline and world == 1:
        times, threads = oracle_sample(wl, 5, 1)
        cus = 1e6 * sum(times) / len(times)
        out["cpu_baseline"] = {"value": cus, "unit": "us", "cores": threads, "kind": "oracle",
                               "sample": f"{len(times)} verify steps of stream 0 ({R} rows, prefix "
                                         f"{wl.prefix_lens[0]}, synthetic K/V), float64 numpy"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--beta", type=float, default=0.4)
    ap.add_argument("--gamma", type=int, default=None, help="draft length (config 2's sweep)")
    ap.add_argument("--prefix", type=int, default=None, help="prefix length (config 2's sweep)")
    ap.add_argument("--draft-noise", type=float, default=1.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--beta-sweep", action="store_true",
                    help="run the loop at beta = 0, 0.1 .. 0.4 (the sweep of the paper's Table 3, cost side)")
    ap.add_argument("--loop-iterations", type=int, default=200,
                    help="SSD iterations timed for the tokens/s figure (0: skip the loop)")
    ap.add_argument("--synthetic-kv", action="store_true",
                    help="seed the prefix K/V with noise instead of running a prefill (short profiling runs)")
    ap.add_argument("--print-kernel-hash", action="store_true",
                    help="print the hash of the persistent kernel's sources (for a profile summary) and exit")
    args = ap.parse_args()
    if args.print_kernel_hash:
        print(kernel_sources_sha1())
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
