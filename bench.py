"""Benchmark of the NAV verify pass: verified tokens/s and verify-pass latency, 7B shape, k=8.

One step = one speculative round through the public C ABI: pipesd_verify (target forward over the
pending token + k drafts against the cached prefix, accept/correct rule) + pipesd_ctx_sync (the two
result ints come back to the host) + pipesd_kv_rollback.  The cache grows by n_accepted+1 per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 7b-k8]

Prints ONE JSON line (rank 0).  Multi-GPU runs are independent replicas (no collective on the path).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from paper_2605_13319_b200 import synth  # noqa: E402

WORKLOADS = {
    # name: (shape, prefix, k, sigma)
    "7b-k8": ("7b", 2048, 8, 1.0),
    "7b-k4": ("7b", 2048, 4, 1.0),
    "7b-k16": ("7b", 2048, 16, 1.0),
    "1b-k8": ("1b", 512, 8, 1.0),
    "8b-k16": ("8b", 8192, 16, 0.5),
    "tiny-k4": ("tiny", 64, 4, 1.0),
    "7b2l-k8": ("7b2l", 2048, 8, 1.0),   # two layers of the 7b shape: small enough for counter captures
}
METRIC = "verified tokens/sec (verify-pass latency in ms_per_step), k=8, 7B shape, % of HBM roofline"
NOMINAL_HBM_GBS = 8000.0


def peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def pass_bytes(shape, k, cached_len):
    """Algorithmic bytes of one verify pass: every weight once (bf16), embedding rows of the k+1 tokens,
    K/V of the cached prefix read and of the k+1 new rows written, logits written + read once, q read."""
    M = k + 1
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab
    per_layer = (shape.q_dim + 2 * shape.kv_dim) * d + d * shape.q_dim + 3 * F * d
    weights = 2 * (shape.n_layers * per_layer + V * d) + 4 * d * (2 * shape.n_layers + 1) + 2 * M * d
    kv_tok = 2 * shape.n_layers * shape.kv_dim * 2
    kv = kv_tok * (cached_len + M)
    vocab_io = 4 * M * V * 2 + 4 * k * V
    return weights + kv + vocab_io


class ClockSampler:
    """nvidia-smi samples of the SM clock and throttle reasons while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "50"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 8:
                continue
            try:
                sm.append(float(c[0])); mx.append(float(c[1]))
            except ValueError:
                continue
            for n, v in zip(names, c[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def draw_from(q_row, u):
    cdf = np.cumsum(q_row.astype(np.float64))
    return min(int(np.searchsorted(cdf, float(u) * cdf[-1], side="right")), q_row.size - 1)


def softmax64(x):
    x = x.astype(np.float64)
    e = np.exp(x - x.max())
    return e / e.sum()


def record_rounds(ctx, req, shape, k, sigma, seed, n_rounds, torch):
    """Untimed: produce every round's inputs by running the target one token at a time through the
    library (q_i = softmax(target logits + sigma*noise), draft ~ q_i), then verify + rollback so that
    the next round starts from the committed state.  Returns the per-round inputs and outcomes."""
    from paper_2605_13319_b200 import binding
    V = shape.vocab
    rounds = []
    pending = synth.make_pending(shape, seed)
    for r in range(n_rounds):
        base = ctx.req_len(req)
        noise = synth.normal_f32((k, V), seed, synth.STREAM_NOISE + 7919 * r)
        du = synth.uniform_f32(k, seed, synth.STREAM_DRAFT_U + 7919 * r)
        toks = [int(pending)]
        q = np.empty((k, V), np.float32)
        for i in range(k):
            l = ctx.prefill(req, [toks[-1]], want_last_logits=True)
            q[i] = softmax64(l.astype(np.float64) + sigma * noise[i]).astype(np.float32)
            toks.append(draw_from(q[i], du[i]))
        ctx.debug_set_len(req, base)
        toks = np.array(toks, np.int32)
        u = synth.make_accept_uniforms(k, seed, 0, r)
        q_dev = torch.from_numpy(q).to(ctx.device)
        q_pin = torch.from_numpy(q).pin_memory()
        ((n_acc, nxt),) = ctx.verify([dict(req=req, tokens=toks, q=q_dev, u=u)])
        ctx.kv_rollback([req], [n_acc])
        rounds.append(dict(tokens=toks, q_dev=q_dev, q_pin=q_pin, u=u, n_acc=n_acc, next=nxt, base=base))
        pending = nxt
    return rounds


def replay(ctx, req, rounds, host_q, torch, timed=True):
    """Run recorded rounds back to back, bracketed by CUDA events on the context's stream when timed.
    Returns (elapsed_ms, verified tokens, results that differ from the recording)."""
    from paper_2605_13319_b200 import binding
    st = ctx.stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tokens = mism = 0
    torch.cuda.synchronize()
    e0.record(st)
    for rd in rounds:
        if host_q:
            item = dict(req=req, tokens=rd["tokens"], q=rd["q_pin"].numpy(), u=rd["u"])
            ((n_acc, nxt),) = ctx.verify([item], flags=binding.Q_HOST)
        else:
            ((n_acc, nxt),) = ctx.verify([dict(req=req, tokens=rd["tokens"], q=rd["q_dev"], u=rd["u"])])
        ctx.kv_rollback([req], [rd["n_acc"]])   # the recorded decision keeps the trajectory fixed
        mism += (n_acc, nxt) != (rd["n_acc"], rd["next"])
        tokens += rd["n_acc"] + 1
    e1.record(st)
    torch.cuda.synchronize()
    return (e0.elapsed_time(e1) if timed else 0.0), tokens, mism


def oracle_sample(shape, weights, P, k, sigma, seed, n_layers=None):
    """Time the CPU checker's verify call (as it stands) on one round of the workload: synthetic seeded
    K/V prefix of P rows (a CPU prefill is out of reach), its own drafts, then the timed verify."""
    import oracle
    if n_layers is not None and n_layers < shape.n_layers:
        shape = shape.scaled(n_layers=n_layers)
        weights = dict(weights, layers=weights["layers"][:n_layers])
    orc = oracle.Oracle(shape, weights, P + k + 8)
    std = 0.02 * np.sqrt(shape.d_model)
    for l in range(shape.n_layers):
        kk, vv = synth.make_synthetic_kv(shape, P, seed, l, std_k=std, std_v=std)
        orc.set_synthetic_kv(l, kk, vv)
    orc.set_len(P)
    V = shape.vocab
    toks, q, _ = orc.draft_round(synth.make_pending(shape, seed), k, sigma,
                                 synth.normal_f32((k, V), seed, synth.STREAM_NOISE),
                                 synth.uniform_f32(k, seed, synth.STREAM_DRAFT_U))
    u = synth.make_accept_uniforms(k, seed)
    t0 = time.perf_counter()
    r = orc.verify(toks, q, u)
    dt = time.perf_counter() - t0
    return dt, r["n_accepted"] + 1, orc


def run_reference(args, shape, P, k, sigma):
    """--impl reference: the CPU checker timed on the host cores, each step a bounded sample."""
    cores = os.cpu_count() or 1
    steps, warm = args.steps, args.warmup
    budget = 150.0
    # one layer + head first, to size the sample
    w1 = synth.make_weights(shape.scaled(n_layers=1), 0)
    t1, _, _ = oracle_sample(shape.scaled(n_layers=1), w1, P, k, sigma, 0)
    est_full = t1 * shape.n_layers
    nl = int(max(1, min(shape.n_layers, budget / max(1e-9, (steps + warm) * est_full) * shape.n_layers)))
    sh = shape.scaled(n_layers=nl)
    w = synth.make_weights(sh, 0)
    import oracle
    orc = oracle.Oracle(sh, w, P + k + 8)
    std = 0.02 * np.sqrt(shape.d_model)
    for l in range(nl):
        kk, vv = synth.make_synthetic_kv(sh, P, 0, l, std_k=std, std_v=std)
        orc.set_synthetic_kv(l, kk, vv)
    orc.set_len(P)
    V = shape.vocab
    toks, q, _ = orc.draft_round(synth.make_pending(shape, 0), k, sigma,
                                 synth.normal_f32((k, V), 0, synth.STREAM_NOISE),
                                 synth.uniform_f32(k, 0, synth.STREAM_DRAFT_U))
    u = synth.make_accept_uniforms(k, 0)
    total, tokens = 0.0, 0
    for s in range(steps + warm):
        t0 = time.perf_counter()
        r = orc.verify(toks, q, u)
        dt = time.perf_counter() - t0
        orc.truncate(P)
        if s >= warm:
            total += dt
            tokens += r["n_accepted"] + 1
    scale = shape.n_layers / nl
    ms = total / steps * scale * 1e3
    value = tokens / (total * scale)
    sample = (f"oracle verify pass on {nl} of {shape.n_layers} layers + LM head per step (time scaled by "
              f"{scale:.2f}), synthetic seeded K/V prefix of {P} rows, one fixed round of drafts")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape.name, "prefix": P, "k": k, "sigma": sigma},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b-k8", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--engine", default="tiled", choices=["tiled", "persistent"],
                    help="which kernels run the layer stack (the headline is the faster one on this workload: tiled)")
    ap.add_argument("--no-other-engine", action="store_true", help="skip the short timing of the other engine")
    ap.add_argument("--quick-inputs", action="store_true",
                    help="profiler runs: seeded synthetic K/V prefix and random drafts instead of a recorded "
                         "trajectory, one timed region only, so that few launches precede the captured ones")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    sname, P, k, sigma = WORKLOADS[args.workload]
    shape = synth.B7.scaled(name="7b2l", n_layers=2) if sname == "7b2l" else synth.SHAPES[sname]
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, shape, P, k, sigma)
        return

    import torch
    import torch.distributed as dist
    from paper_2605_13319_b200 import binding, build
    build.build_cuda()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    seed = 0
    n_rounds = args.warmup + args.steps
    max_seq = P + n_rounds * (k + 1) + 64
    weights = synth.make_weights(shape, seed)
    ctx = binding.Context(shape, weights, n_pages=max_seq // 16 + 4, max_seq=max_seq, max_draft=max(k, 16),
                          device=local, engine=args.engine)
    prefix = synth.make_prefix(shape, P, seed + rank)
    if args.quick_inputs:
        quick_run(args, ctx, shape, P, k, seed, torch)
        return

    def fresh():
        req = ctx.req_open()
        ctx.prefill(req, prefix)
        return req

    req = fresh()
    rounds = record_rounds(ctx, req, shape, k, sigma, seed, n_rounds, torch)
    ctx.req_close(req)

    uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    sampler = ClockSampler(uuid)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()

    # -- timed region 1: inputs resident in HBM
    req = fresh()
    ctx.profile_enable(False)
    barrier()
    sampler.start()
    replay(ctx, req, rounds[:args.warmup], False, torch, timed=False)  # warm-up
    ctx.profile_read()
    ms, tokens, mism = replay(ctx, req, rounds[args.warmup:], False, torch)
    prof = ctx.profile_read()
    barrier()
    ctx.req_close(req)
    # -- timed region 2: host buffers (q copied H2D inside, results D2H)
    req = fresh()
    replay(ctx, req, rounds[:args.warmup], True, torch, timed=False)
    barrier()
    ms_e2e, tokens_e2e, mism2 = replay(ctx, req, rounds[args.warmup:], True, torch)
    barrier()
    ctx.req_close(req)
    # -- region 3: the same steps with every weight-streaming GEMM launch bracketed by CUDA events
    req = fresh()
    replay(ctx, req, rounds[:args.warmup], False, torch, timed=False)
    ctx.profile_enable(True)
    ms_prof, _, _ = replay(ctx, req, rounds[args.warmup:], False, torch)
    gprof = ctx.profile_read()
    ctx.profile_enable(False)
    ctx.req_close(req)
    # -- the other engine on the same recorded rounds (device-resident inputs only), for comparison
    other = None
    if world == 1 and not args.no_other_engine:
        ctx.close()
        oname = "persistent" if args.engine == "tiled" else "tiled"
        ctx = binding.Context(shape, weights, n_pages=max_seq // 16 + 4, max_seq=max_seq, max_draft=max(k, 16),
                              device=local, engine=oname)
        req = ctx.req_open()
        ctx.prefill(req, prefix)
        replay(ctx, req, rounds[:args.warmup], False, torch, timed=False)
        ctx.profile_enable(False)
        ctx.profile_read()
        ms_o, tokens_o, mism_o = replay(ctx, req, rounds[args.warmup:], False, torch)
        prof_o = ctx.profile_read()
        other = {"engine": oname, "ms_per_step": ms_o / args.steps, "value": tokens_o / (ms_o * 1e-3), "unit": "tokens/s",
                 "gpu_launches": int(prof_o["kernel_launches"]),
                 "decisions_differing_from_recording": int(mism_o)}
        ctx.req_close(req)
    clocks = sampler.stop()

    # -- reduce over ranks: max time, summed tokens
    if world > 1:
        from paper_2605_13319_b200 import replicas
        (ms, ms_e2e), (tokens, tokens_e2e) = replicas.reduce_replicas([ms, ms_e2e], [tokens, tokens_e2e], device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    steps = args.steps
    ms_step = ms / steps
    bytes_pass = float(np.mean([pass_bytes(shape, k, rd["base"]) for rd in rounds[args.warmup:]]))
    peak, peak_kind = peaks()
    gemm_gbs = gprof["gemm_bytes"] / (gprof["gemm_ms"] * 1e-3) / 1e9 if gprof["gemm_ms"] > 0 else 0.0
    line = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 weights x split-bf16 activations, fp32 accumulate", "data": "synthetic",
        "config": {"workload": args.workload, "shape": shape.name, "prefix": P, "k": k, "sigma": sigma, "engine": args.engine,
                   "rounds": steps, "l2": "inputs larger than L2 (weights streamed once per pass)",
                   "accepted_per_step": tokens / world / steps - 1.0, "replay_mismatches": int(mism + mism2)},
        "pass": {"bytes": bytes_pass, "gbs": bytes_pass / (ms_step * 1e-3) / 1e9,
                 "frac_of_nominal_8TBs": bytes_pass / (ms_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                 "frac_of_measured_copy": bytes_pass / (ms_step * 1e-3) / 1e9 / peak},
        "e2e": {"value": tokens_e2e / (ms_e2e * 1e-3), "unit": "tokens/s", "ms_per_step": ms_e2e / steps,
                "h2d_bytes_per_step": int(4 * k * shape.vocab + 4 * (k + 1) * 2),
                "d2h_bytes_per_step": 16},
        "gpu_launches": int(prof["kernel_launches"]),
        "roofline": {"bound": "hbm", "kernel": "gemm_wstream_kernel" if args.engine == "tiled" else "mega_kernel", "achieved": gemm_gbs, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": gemm_gbs / peak,
                     "launches": int(gprof["gemm_launches"]), "share_of_step": gprof["gemm_ms"] / ms_prof,
                     "ms_per_step_with_events": ms_prof / steps,
                     "algorithmic_bytes_per_launch": gprof["gemm_bytes"] / max(1, gprof["gemm_launches"]),
                     "traffic": TRAFFIC_7B_K8.get(args.engine) if args.workload == "7b-k8" else None},
        "clocks": clocks,
    }
    if other is not None:
        line["other_engine"] = other
    if world == 1 and not args.no_cpu_baseline:
        dt, toks_o, _ = oracle_sample(shape, weights, P, k, sigma, seed)
        line["cpu_baseline"] = {"value": toks_o / dt, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
                                "ms_per_pass": dt * 1e3,
                                "sample": f"one verify pass (all {shape.n_layers} layers, k={k}) against a seeded "
                                          f"synthetic K/V prefix of {P} rows, drafts made by the oracle itself"}
    print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def quick_run(args, ctx, shape, P, k, seed, torch):
    """Profiler-friendly variant: no prefill passes, no recording.  Kernel durations do not depend on the
    values, only on the shapes and lengths, which are those of the workload."""
    V = shape.vocab
    req = ctx.req_open()
    std = 0.02 * np.sqrt(shape.d_model)
    for l in range(shape.n_layers):
        kk, vv = synth.make_synthetic_kv(shape, P, seed, l, std_k=std, std_v=std)
        ctx.debug_write_kv(req, l, 0, kk, vv)
    rounds = []
    for r in range(args.warmup + args.steps):
        noise = synth.normal_f32((k, V), seed, synth.STREAM_NOISE + 7919 * r)
        q = np.stack([softmax64(noise[i]) for i in range(k)]).astype(np.float32)
        toks = synth.tokens_i32(k + 1, seed, synth.STREAM_PENDING + r, V)
        rounds.append(dict(tokens=toks, q_dev=torch.from_numpy(q).to(ctx.device), u=synth.make_accept_uniforms(k, seed, 0, r)))
    st = ctx.stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tokens = 0
    for i, rd in enumerate(rounds):
        if i == args.warmup:
            torch.cuda.synchronize()
            e0.record(st)
        ((n_acc, nxt),) = ctx.verify([dict(req=req, tokens=rd["tokens"], q=rd["q_dev"], u=rd["u"])])
        ctx.kv_rollback([req], [n_acc])
        tokens += (n_acc + 1) if i >= args.warmup else 0
    e1.record(st)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    print(json.dumps({"mode": "quick-inputs", "workload": args.workload, "steps": args.steps, "warmup": args.warmup,
                      "ms_per_step": ms / args.steps, "tokens": tokens}), flush=True)
    ctx.close()


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised
# under profiles/ (taken on a two-layer model of the same shape -- same per-layer work -- and scaled to a full
# launch by the layers it covers).  None until a capture of the current kernel exists, and to be reset to None
# whenever that kernel changes.
TRAFFIC_7B_K8 = {"tiled": 103.0e6, "persistent": 14.37e9}


if __name__ == "__main__":
    main()
