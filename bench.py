#!/usr/bin/env python
"""Benchmark of the verify step (one pass of the whole hot path over one batch of synthetic input).

    python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]

Prints ONE JSON line.  `value` is verified tokens per second (rows pushed through verification per
second, whole job) with the step's inputs resident in device memory; `e2e` is the same metric through
the public ts_verify call with host buffers (inputs copied host->device and results device->host
inside the timed region).  Multi-GPU runs are independent replicas (the path has no exchange step).
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# name -> (shape, [context lengths], [k per sequence])
WORKLOADS = {
    "c1_tiny_ctx256_k8": ("tiny", [256], [8]),
    "c2_1b_ctx4096_k4": ("1b", [4096], [4]),
    "c2_1b_ctx4096_k8": ("1b", [4096], [8]),
    "c2_1b_ctx4096_k16": ("1b", [4096], [16]),
    "c3_8b_ctx2048_k32": ("8b", [2048], [32]),
    "c3_8b_ctx8192_k1": ("8b", [8192], [1]),
    "c3_8b_ctx8192_k4": ("8b", [8192], [4]),
    "c3_8b_ctx8192_k8": ("8b", [8192], [8]),
    "c3_8b_ctx8192_k16": ("8b", [8192], [16]),
    "c3_8b_ctx8192_k32": ("8b", [8192], [32]),
    "c5_8b_b4_ctx8192_k64": ("8b", [8192] * 4, [64] * 4),
    # reduced-depth case for profiler captures (same per-layer kernels and grids as c3)
    "prof_8b4l_ctx8192_k32": ("8b-4l", [8192], [32]),
    "prof_8b4l_b4_ctx2048_k64": ("8b-4l", [2048] * 4, [64] * 4),
}
DEFAULT_WORKLOAD = "c3_8b_ctx8192_k32"
METRIC = "verified_tokens_per_s"
UNIT = "tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the projection GEMM, from the ncu
# capture summarised under profiles/ (None until a capture exists)
GEMM_TRAFFIC_BYTES_PER_LAUNCH = 107.1e6    # (36 x 396.2 MB measured per layer + the LM-head launch by its algorithmic bytes) / 145 launches
# the same for one launch of the persistent kernel on the default workload
FUSED_TRAFFIC_BYTES_PER_LAUNCH = None


def c4_workload():
    """Config 4: 16 sessions, contexts log-uniform over 2k..16k, k uniform in 4..32 (seeded)."""
    import numpy as np
    g = np.random.Generator(np.random.Philox(key=[260413519, 4]))
    lens = [int(round(2048 * 8 ** float(u))) for u in g.random(16)]
    ks = [int(x) for x in g.integers(4, 33, size=16)]
    return "8b", lens, ks


def get_workload(name):
    if name == "c4_8b_b16_ragged":
        return c4_workload()
    return WORKLOADS[name]


def algorithmic_bytes(shape, lens, ks):
    """Bytes one verify step must move: every weight matrix once, the context K/V once, the chunk's
    K/V written, the logits written, the embedding rows read (the embedding table itself is not)."""
    s = shape
    M = sum(ks)
    weights = 2 * s.n_params_matmul()
    kv_read = sum(lens) * 4 * s.n_kv_heads * s.head_dim * s.n_layers
    kv_write = M * 4 * s.n_kv_heads * s.head_dim * s.n_layers
    return dict(weights=weights, kv_read=kv_read, kv_write=kv_write, logits=4 * M * s.vocab,
                embed=2 * M * s.d_model,
                total=weights + kv_read + kv_write + 4 * M * s.vocab + 2 * M * s.d_model)


def algorithmic_flops(shape, lens, ks):
    s = shape
    M = sum(ks)
    attn = sum(4 * s.n_q_heads * s.head_dim * s.n_layers * k * (n + k / 2) for n, k in zip(lens, ks))
    return 2 * M * s.n_params_matmul() + attn


def gemm_bytes_per_step(shape, M, planes):
    """Algorithmic bytes of the projection-GEMM launches of one step and their count: each weight
    matrix once plus the activation rows in and the result rows out."""
    s = shape
    d, F, Nq, Nkv = s.d_model, s.d_ffn, s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    per_layer = [((Nq + 2 * Nkv), d, 4), (d, Nq, 4), (2 * F, d, 1 * planes), (d, F, 4)]   # (N, K, out bytes per (m, n) / 2 for swiglu)
    total = 0
    for N, K, ob in per_layer:
        out = M * N * 4 if ob == 4 else M * (N // 2) * 2 * planes
        total += N * K * 2 + M * K * 2 * planes + out
    total *= s.n_layers
    total += s.vocab * d * 2 + M * d * 2 * planes + M * s.vocab * 4
    return total, 4 * s.n_layers + 1


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=j["hbm_gbs"], bf16_tflops=j.get("bf16_tflops_sustained", j["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.rows, self.proc = uuid, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=mx, reasons=sorted(reasons),
                    samples=len(sm))


def tree_parents(k):
    """Parent node of each of the k - 1 draft nodes: four chains hanging from the root (node 0), of about
    1/2, 1/4, 1/8 and 1/8 of the drafts -- the proportions of the 32/16/8/8 continuation lengths."""
    n = k - 1
    lens = [n - n // 2, n // 2 - n // 4, n // 4 - n // 8, n // 8]
    par, node = [], 1
    for ln in lens:
        for j in range(ln):
            par.append(0 if j == 0 else node - 1)
            node += 1
    assert len(par) == n
    return par


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value_ms: float, world: int, backend_device=None) -> float:
    """Slowest rank's time (replicas run independently; the job's time is the maximum)."""
    if world == 1:
        return value_ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([value_ms], dtype=torch.float64, device=backend_device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def build_gpu_model(shape, lens, ks, act_split=True, path=0):
    """Random-init weights generated on the device (N(0, 0.02) rounded to bf16, gains one) and a KV
    pool filled with N(0,1) fp16 values; sessions placed at their context lengths."""
    import torch
    import paper_2604_13519_b200 as ts
    from paper_2604_13519_b200 import binding as B
    B_, k_max = len(lens), max(max(ks), 8)
    max_ctx = max(lens) + 2 * k_max
    pages = sum((n + 2 * k_max + 15) // 16 for n in lens) + 8
    m = ts.Model(shape, max_pages=pages, max_batch=B_, k_max=k_max, max_rows=max(sum(ks), k_max),
                 max_ctx=max_ctx, act_split=act_split, path=path)
    g = torch.Generator(device="cuda").manual_seed(260413519)
    s = shape

    def rnd(r, c):
        return (torch.randn(r, c, generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
    ones = torch.ones(s.d_model, dtype=torch.float32, device="cuda")
    m.load_tensor(B.TS_W_EMBED, 0, rnd(s.vocab, s.d_model))
    m.load_tensor(B.TS_W_LM_HEAD, 0, rnd(s.vocab, s.d_model))
    m.load_tensor(B.TS_W_FINAL_GAIN, 0, ones)
    Nq, Nkv = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    for l in range(s.n_layers):
        m.load_tensor(B.TS_W_Q, l, rnd(Nq, s.d_model))
        m.load_tensor(B.TS_W_K, l, rnd(Nkv, s.d_model))
        m.load_tensor(B.TS_W_V, l, rnd(Nkv, s.d_model))
        m.load_tensor(B.TS_W_O, l, rnd(s.d_model, Nq))
        m.load_tensor(B.TS_W_GATE, l, rnd(s.d_ffn, s.d_model))
        m.load_tensor(B.TS_W_UP, l, rnd(s.d_ffn, s.d_model))
        m.load_tensor(B.TS_W_DOWN, l, rnd(s.d_model, s.d_ffn))
        m.load_tensor(B.TS_W_GAIN1, l, ones)
        m.load_tensor(B.TS_W_GAIN2, l, ones)
    kv = m.kv_pool_tensor()
    step = 1 << 28
    for i in range(0, kv.numel(), step):
        kv[i:i + step].normal_(generator=g)
    sessions = []
    for n in lens:
        ss = ts.Session(m, None, None)
        ss.set_cache(n, 3)
        sessions.append(ss)
    torch.cuda.synchronize()
    return m, sessions


def oracle_sample_seconds(shape, lens, ks, n_layers_sample):
    """Time the CPU oracle on the same chunk over the first n_layers_sample layers plus the LM head,
    then scale the per-layer part to the full depth.  Returns (seconds for a full step, threads)."""
    import torch
    import oracle
    import synth
    layers = list(range(min(n_layers_sample, shape.n_layers)))
    sub = synth.ModelShape(**{**shape.asdict(), "n_layers": len(layers), "name": shape.name + "-sample"})
    w = synth.make_weights(shape, layers=layers)
    om = oracle.OracleModel(sub, w)
    t_layers = 0.0
    t_head = 0.0
    for i, (n, k) in enumerate(zip(lens, ks)):
        K, V = synth.make_synthetic_kv(sub, n, stream=i)
        cache = om.new_cache()
        cache.import_kv(K, V)
        toks = [3] + [64 + j for j in range(k - 1)]
        t0 = time.perf_counter()
        x = om.w["embed"][torch.tensor(toks)].to(torch.float64)
        pos = torch.arange(k) + n
        for l in range(len(layers)):
            x, _, _ = om._layer(l, x, pos, cache.k[l], cache.v[l], torch.arange(n))
        t1 = time.perf_counter()
        logits = om._head(x)
        oracle.argmax_lowest(logits)
        t2 = time.perf_counter()
        t_layers += t1 - t0
        t_head += t2 - t1
    full = t_layers * shape.n_layers / len(layers) + t_head
    return full, torch.get_num_threads(), len(layers)


def run_reference(args, shape, lens, ks, name):
    """Reference arm: the CPU oracle, as it stands, on the host cores; each step a bounded sample."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    n_sample = 2 if shape.n_layers > 4 else shape.n_layers
    times = []
    for i in range(args.warmup + args.steps):
        sec, threads, nl = oracle_sample_seconds(shape, lens, ks, n_sample)
        if i >= args.warmup:
            times.append(sec)
    ms = 1e3 * sum(times) / len(times)
    value = sum(ks) / (ms / 1e3)
    sample = f"chunk forward over the first {nl} of {shape.n_layers} layers + LM head, layer time scaled to full depth"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": name, "batch": len(lens), "context": lens, "k": ks},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_retrieval(args, shape):
    """Top-K of Eq. 3 over N seeded N(0,1) hidden states (bf16), K = 10: one pass over N x d x 2 bytes."""
    import torch
    import paper_2604_13519_b200 as ts
    tiny = ts.Model(shape if shape.n_layers <= 4 else __import__("synth").SHAPES[shape.name + "-2l"], max_pages=8, max_batch=1,
                    k_max=8, max_rows=8, max_ctx=64, act_split=True, path=1)
    d, N = shape.d_model, args.retrieval
    g = torch.Generator(device="cuda").manual_seed(260413519)
    H = torch.randn(N, d, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    q = torch.randn(d, generator=g, device="cuda", dtype=torch.float32)
    for _ in range(max(args.warmup, 3)):
        ts.ts_topk_cosine(tiny, H, 10, query=q)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ts.ts_topk_cosine(tiny, H, 10, query=q)
    torch.cuda.synchronize()
    ms = 1e3 * (time.perf_counter() - t0) / args.steps
    peaks = measured_peaks()
    gbs = N * d * 2 / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "topk_cosine_ms", "value": ms, "unit": "ms", "n_gpus": 1, "steps": args.steps,
                      "warmup": max(args.warmup, 3), "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
                      "config": {"workload": f"retrieval over {N} hidden states of width {d}, K = 10",
                                 "timing": "host clock around the public call (launches, result copy, stream sync)"},
                      "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"]}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sweep", action="store_true", help="skip the latency-vs-k sweep")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-act-split", action="store_true")
    ap.add_argument("--path", type=int, default=0, help="0 auto, 1 one kernel per stage, 2 single persistent kernel")
    ap.add_argument("--retrieval", type=int, default=0,
                    help="N > 0: time ts_topk_cosine (K = 10) over N synthetic hidden states of the workload's width "
                         "instead of the verify step, and print its own JSON line")
    ap.add_argument("--want-topk", action="store_true",
                    help="also take the per-position Top-K of the logits (TS_FLAG_WANT_TOPK), as the recycling drafter needs")
    ap.add_argument("--temperature", type=float, default=0.0,
                    help="> 0: speculative-sampling acceptance at this temperature (ts_verify_sampled) with fixed uniforms")
    ap.add_argument("--tree", action="store_true",
                    help="verify each chunk as a draft tree (four branches from the root, lengths about 1/2, 1/4, 1/8, "
                         "1/8 of the drafts: the shape of the retrieval candidate set) through ts_verify_tree")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    import synth
    shape_name, lens, ks = get_workload(args.workload)
    shape = synth.SHAPES[shape_name]
    if args.impl == "reference":
        run_reference(args, shape, lens, ks, args.workload)
        return

    import torch
    import paper_2604_13519_b200 as ts
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verify path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if args.retrieval > 0:
        run_retrieval(args, shape)
        return
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    ts.binding.lib()
    planes = 1 if args.no_act_split else 2
    model, sessions = build_gpu_model(shape, lens, ks, act_split=not args.no_act_split, path=args.path)
    M = sum(ks)
    drafts = [[64 + (7 * j + i) % (shape.vocab - 64) for j in range(k - 1)] for i, k in enumerate(ks)]
    stream = torch.cuda.current_stream()
    parents = [tree_parents(k) for k in ks] if args.tree else None

    uniforms = [((37 * r + 11) % 100) / 100.0 for r in range(M)]

    vflags = ts.TS_FLAG_WANT_TOPK if args.want_topk else 0

    def verify():
        if args.temperature > 0:
            return ts.ts_verify_sampled(model, sessions, drafts, args.temperature, uniforms, flags=vflags)
        if parents is None:
            return ts.ts_verify(model, sessions, drafts, flags=vflags)
        return ts.ts_verify_tree(model, sessions, drafts, parents, flags=vflags)

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    # ---- e2e arm: the public call with host buffers --------------------------------------------
    for _ in range(args.warmup):
        verify()
    l0, h0, d0 = model.counters()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        verify()
    torch.cuda.synchronize()
    e2e_ms = 1e3 * (time.perf_counter() - t0) / args.steps
    l1, h1, d1 = model.counters()
    launches_per_step = (l1 - l0) // args.steps
    e2e_ms = max_over_ranks(e2e_ms, world, "cuda")

    # ---- device-resident arm: replay the staged step ---------------------------------------------
    for _ in range(args.warmup):
        ts.ts_verify_replay(model)
    uuid = str(torch.cuda.get_device_properties(local_rank).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        ts.ts_verify_replay(model)
    ev1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1) / args.steps
    ms = max_over_ranks(ms, world, "cuda")

    # ---- per-step latency distribution and the per-kernel pass -------------------------------------
    lat = []
    for _ in range(min(args.steps, 50)):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ts.ts_verify_replay(model)
        b.record(stream)
        b.synchronize()
        lat.append(a.elapsed_time(b))
    prof = {}
    for _ in range(3):
        p = ts.ts_profile_step(model)
        for kcls, (pm, pn) in p.items():
            a = prof.setdefault(kcls, [0.0, 0])
            a[0] += pm / 3
            a[1] = pn
    peaks = measured_peaks()
    ab = algorithmic_bytes(shape, lens, ks)
    fl = algorithmic_flops(shape, lens, ks)
    t_hbm = ab["total"] / (peaks["hbm_gbs"] * 1e9)
    t_tc = fl / (peaks["bf16_tflops"] * 1e12)
    bound = "hbm" if t_hbm >= t_tc else "tensor"
    fused_ms, fused_n = prof.get("fused_kernel", (0.0, 0))
    if fused_n:
        # the step is ONE launch of the persistent kernel: its algorithmic bytes are the step's; its
        # duration is the average launch duration over the timed region (launches run back to back)
        gbs = ab["total"] / (ms * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "fused_verify_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": FUSED_TRAFFIC_BYTES_PER_LAUNCH,
                    "peak_source": peaks["source"], "bytes_per_launch": ab["total"], "ms_per_launch": ms,
                    "phase_ms": {k: v[0] for k, v in prof.items() if k in ("gemm", "attention", "attention_merge")}}
    else:
        gemm_bytes, gemm_launches = gemm_bytes_per_step(shape, M, planes)
        gemm_ms, gemm_n = prof["gemm"]
        gemm_gbs = gemm_bytes / gemm_launches / (gemm_ms / gemm_n * 1e-3) / 1e9 if gemm_n else None
        roofline = {"bound": "hbm", "kernel": "gemm_ws_kernel", "achieved": gemm_gbs, "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": gemm_gbs / peaks["hbm_gbs"] if gemm_gbs else None,
                    "traffic": GEMM_TRAFFIC_BYTES_PER_LAUNCH, "peak_source": peaks["source"],
                    "bytes_per_launch": gemm_bytes / gemm_launches,
                    "ms_per_launch": gemm_ms / gemm_n if gemm_n else None}
    step_roof = {"bound": bound, "bytes": ab["total"], "flops": fl, "achieved_gbs": ab["total"] / (ms * 1e-3) / 1e9,
                 "frac_of_measured_hbm": ab["total"] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                 "frac_of_nominal_8tbs": ab["total"] / (ms * 1e-3) / 1e9 / 8000.0,
                 "roofline_ms": 1e3 * max(t_hbm, t_tc), "frac": max(t_hbm, t_tc) / (ms * 1e-3)}

    sweep = None
    if not args.no_sweep and len(lens) == 1 and rank == 0:
        sweep = {}
        for k in sorted({1, 4, 8, 16, 32, ks[0]}):
            if k > model.cfg.k_max:
                continue
            ts.ts_verify(model, sessions, [drafts[0][:k - 1]])
            for _ in range(3):
                ts.ts_verify_replay(model)
            ls = []
            for _ in range(20):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                ts.ts_verify_replay(model)
                b.record(stream)
                b.synchronize()
                ls.append(a.elapsed_time(b))
            sweep[str(k)] = {"p50_ms": statistics.median(ls), "verified_tok_s": k / (statistics.median(ls) * 1e-3)}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_sample = 4 if shape.n_layers > 8 else shape.n_layers
        sec, threads, nl = oracle_sample_seconds(shape, lens, ks, n_sample)
        cpu = {"value": M / sec, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"one chunk forward over the first {nl} of {shape.n_layers} layers + LM head on the same "
                         f"shapes, layer time scaled to full depth ({sec:.1f} s per step)"}

    if rank == 0:
        out = {
            "metric": METRIC, "value": world * M / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "batch": len(lens), "context": lens, "k": ks,
                       "act_split": planes == 2, "draft_tree": bool(args.tree), "temperature": args.temperature, "per_position_topk": bool(args.want_topk), "kv_dtype": "f16", "l2": "inputs (weights) far larger than L2",
                       "parallelism": "replicas" if world > 1 else "single"},
            "latency_ms": {"p50": statistics.median(lat), "p90": sorted(lat)[int(0.9 * (len(lat) - 1))]},
            "clocks": clocks,
            "e2e": {"value": world * M / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": (h1 - h0) // args.steps, "d2h_bytes_per_step": (d1 - d0) // args.steps},
            "gpu_launches": launches_per_step * args.steps,
            "launches_per_step": launches_per_step,
            "roofline": roofline, "step_roofline": step_roof,
            "kernel_ms_per_step": {k: v[0] for k, v in prof.items()},
            "latency_vs_k": sweep, "cpu_baseline": cpu,
        }
        print(json.dumps(out))
    model.close()
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
