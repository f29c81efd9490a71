"""Decode-throughput benchmark of the q4decode library (one JSON line on stdout).

A step is one decode step of the whole batch (every kernel of the path).  The default workload is the
Qwen3-8B-shaped model at batch 16 with KV lengths drawn log-uniformly from [256, 8192] and four requests
leaving and four joining (512 prefilled tokens) every 32 steps; `--workload` selects the other shapes.

  value      tokens/s with everything resident in HBM (tokens chained on the device, no host sync)
  e2e        tokens/s through q4d_decode_step_host: host inputs, host outputs, a sync per step
  roofline   the dominant kernel (the kernel whose launches take the largest share of the step; the projection
             kernel serves four launch classes per layer) timed with CUDA events around each of its launches
  cpu_baseline  the CPU oracle on whole steps of the same workload, on the host cores
  parity     the last step of the run compared with the oracle (free-running through every layer)

`--impl reference` times the CPU oracle alone (the only reference implementation there is).
With N > 1 every rank runs an independent replica (requests are independent; there is no exchange).
"""
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

WORKLOADS = {
    # name: (shape preset, batch, len lo, len hi, log-uniform, churn)
    "qwen3-8b-b16": ("qwen3-8b-shaped", 16, 256, 8192, True, True),
    "qwen3-8b-b1": ("qwen3-8b-shaped", 1, 256, 8192, True, False),
    "qwen3-0.6b-b16": ("qwen3-0.6b-shaped", 16, 128, 2048, False, True),
    "qwen3-0.6b-b1": ("qwen3-0.6b-shaped", 1, 256, 256, False, False),
    "llama-3.2-3b-b16": ("llama-3.2-3b-shaped", 16, 512, 4096, False, False),
    "llama-3.2-3b-b1": ("llama-3.2-3b-shaped", 1, 512, 4096, False, False),
    "moe-30b-b16": ("moe-30b-a3b-shaped", 16, 512, 4096, False, False),
    "moe-30b-b1": ("moe-30b-a3b-shaped", 1, 512, 4096, False, False),
}
METRIC = "decode_tokens_per_second"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu):
        self.rows, self.proc, self.gpu = [], None, gpu

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        good = [(t, r) for t, r in self.rows if len(r) >= 9]
        rows = [r for t, r in good if t0 <= t <= t1] or [r for _, r in good]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(float(r[1]) for r in rows)
        reasons = set()
        for r in rows:
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7),
                              ("sw_power_cap", 8)):
                if r[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": float(rows[0][2]), "reasons": sorted(reasons),
                "samples": len(rows)}


def step_bytes(shape, lens, n, touched=None):
    """Algorithmic bytes of one step: packed weights + scales + biases, KV read and written, logits, embedding rows.
    touched: mixture-of-experts models, the mean number of distinct experts per layer the step routes to (measured:
    q4d_moe_touched_experts); until it is known the expectation under uniform routing stands in."""
    from workload import shapes
    if shape.n_experts and touched is None:
        touched = shape.n_experts * (1.0 - (1.0 - shape.top_k / shape.n_experts) ** n)
    w = shapes.weight_bytes(shape, touched)
    per_tok_layer = 2 * shape.n_kv_heads * shape.head_dim * 2
    kv_read = int(sum(int(l) + 1 for l in lens)) * per_tok_layer * shape.n_layers
    kv_write = n * per_tok_layer * shape.n_layers
    logits = n * shape.vocab * 4
    embed_rows = n * shapes.q4_bytes(1, shape.hidden)
    return {"weights": w, "kv_read": kv_read, "kv_write": kv_write, "logits": logits, "embed": embed_rows,
            "total": w + kv_read + kv_write + logits + embed_rows}


def oracle_steps(shape, weights, pool_t, lens, toks, bt, max_steps, budget_s):
    """Times the oracle, as it stands, on whole decode steps of this workload (every layer, the LM head, the
    argmax): at most max_steps steps, stopping once budget_s seconds are spent.  Every step starts from the same
    pool.  Returns (seconds per step, steps timed, description, threads, (next tokens, logits) of the step)."""
    from oracle import q4d_oracle as orc
    om = orc.OracleModel(shape, weights)
    host_pool = orc.to_np(pool_t).copy()
    times, result = [], None
    while len(times) < max_steps and (not times or sum(times) + times[-1] < budget_s):
        work = host_pool.copy()
        t0 = time.perf_counter()
        nxt, logits, _ = om.decode_step(work, 16, lens, toks, bt)
        times.append(time.perf_counter() - t0)
        result = (nxt, logits)
    desc = (f"{len(times)} whole decode step(s) of this workload (n={len(lens)}, all {shape.n_layers} layers, LM head, "
            f"argmax), {np.mean(times):.2f} s each")
    return float(np.mean(times)), len(times), desc, orc.num_threads(), result


def aggregate_ranks(dist, device, ms, ms_e2e, tokens, tokens_e2e, launches):
    """Replicas only: every rank ran its own batch.  The job's time is the slowest rank's, its tokens and kernel
    launches are the sums over the ranks.  `dist` is torch.distributed with an initialised process group, or None."""
    if dist is None:
        return ms, ms_e2e, tokens, tokens_e2e, launches
    import torch
    t = torch.tensor([ms, ms_e2e], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([tokens, tokens_e2e, launches], dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), int(c[0]), int(c[1]), int(c[2])


def gemm_only(args):
    """One projection shape alone, for kernel-level timing and ncu captures: `--steps` calls of q4d_q4_gemm (operand
    rearrangement + the projection kernel), CUDA events around the loop, one JSON line."""
    import torch

    from paper_2601_19139_b200 import binding as q4d
    from paper_2601_19139_b200 import build as cuda_build
    from workload import gen
    cuda_build.build()
    N, K = (int(v) for v in args.gemm.lower().split("x"))
    n = args.gemm_batch
    torch.cuda.set_device(0)
    ws = [gen.random_q4(N, K, "cuda", "bench-gemm", N, K, i) for i in range(args.gemm_buffers)]
    x = torch.randn((n, K), generator=torch.Generator(device="cpu").manual_seed(args.seed)).to(torch.bfloat16).cuda()
    out = torch.empty(n, N, dtype=torch.float32, device="cuda")
    for i in range(max(args.warmup, 3)):
        q4d.q4_gemm(ws[i % len(ws)], x, n, epilogue=2, out=out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        q4d.q4_gemm(ws[i % len(ws)], x, n, epilogue=2, out=out)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / args.steps
    by = N * K * 0.5625
    peak, kind = peaks()
    print(json.dumps({"op": "q4_gemm", "N": N, "K": K, "n": n, "epilogue": "f32", "calls": args.steps,
                      "kernel": "q4_umma_kernel" if os.environ.get("Q4D_GEMM_KERNEL") == "tcgen05" else "span/round",
                      "us_per_call": us, "GBps": by / us / 1e3, "frac_of_peak": by / us / 1e3 / peak, "peak_kind": kind,
                      "note": "a call = operand rearrangement kernel + projection kernel"}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3-8b-b16", choices=sorted(WORKLOADS))
    ap.add_argument("--profile-steps", type=int, default=8)
    ap.add_argument("--oracle-budget", type=float, default=20.0, help="seconds of oracle steps in the CPU baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--gemm", default=None, metavar="NxK",
                    help="time one 4-bit projection of this shape alone (q4d_q4_gemm, fp32 outputs) instead of the step")
    ap.add_argument("--gemm-batch", type=int, default=16)
    ap.add_argument("--gemm-buffers", type=int, default=1, help="rotate over this many weight tensors (defeats L2)")
    args = ap.parse_args()
    if args.gemm:
        return gemm_only(args)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference" and rank != 0:
        return 0
    if args.warmup < 3:
        args.warmup = 3

    import torch

    from workload import gen, shapes
    preset, n, lo, hi, logu, churn = WORKLOADS[args.workload]
    shape = shapes.PRESETS[preset]
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    dist = None
    if world > 1 and args.impl == "ours":
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    # ---- synthetic model, pool and request script (seeded; the replica of rank k uses seed + k) ----
    seed = args.seed + rank
    weights = gen.make_weights(shape, seed, device)
    total_steps = args.warmup + 2 * args.steps + args.profile_steps + 12
    rng = np.random.default_rng(seed)
    lens0 = gen.draw_lengths(n, lo, hi, rng, logu)
    admits = (total_steps // 32 + 1) * 4 if churn else 0
    blocks = int(sum((l + total_steps + 32) // 16 + 1 for l in lens0) + admits * ((512 + total_steps) // 16 + 2) + 64)
    blocks = max(blocks, int(n * ((hi + total_steps) // 16 + 2)) if n == 1 else blocks)
    pool_t = gen.make_pool(shape, blocks, device)
    script = gen.ChurnScript(shape, pool_t, n, lo, hi, logu, churn_every=32 if churn else 0, churn_count=4,
                             admit_len=512, seed=seed)
    script.prepare_pending(total_steps)
    torch.cuda.synchronize()

    config = {"workload": f"{shape.name}, batch {n}, KV lengths {'log-' if logu else ''}uniform [{lo}, {hi}]"
                          + (", 4 of 16 requests replaced every 32 steps (512 prefilled tokens)" if churn else ""),
              "name": args.workload, "block_size": 16, "weights": "4-bit affine group-64, bf16 scale/bias",
              "l2": "inputs larger than L2 (weights + KV >> 126 MB); no flush needed",
              "layers": shape.n_layers, "hidden": shape.hidden, "vocab": shape.vocab}
    if shape.n_experts:
        config["experts"] = (f"{shape.n_experts} experts, top-{shape.top_k}; weight bytes count the expected number of "
                             f"distinct experts per layer under uniform routing")

    if args.impl == "reference":
        # The reference arm is the CPU oracle on whole steps: one warm-up step, then as many of the requested steps
        # as fit in about two minutes (a step of the 8B shape takes several seconds on the host cores).
        ids, toks, lens, bt = script.step_inputs()
        oracle_steps(shape, weights, pool_t, lens, toks, bt, 1, 0.0)
        t, timed, desc, cores, _ = oracle_steps(shape, weights, pool_t, lens, toks, bt, args.steps, 100.0)
        v = n / t
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s", "n_gpus": 0,
                          "steps": timed, "warmup": 1, "ms_per_step": t * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                           "sample": desc},
                          "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return 0

    from paper_2601_19139_b200 import binding as q4d
    from paper_2601_19139_b200 import build as cuda_build
    cuda_build.build()
    model = q4d.Model(shape, weights, device)
    pool = q4d.KVPool(model, pool_t)
    stream = torch.cuda.current_stream()
    bufs = {"cur": torch.zeros(16, dtype=torch.int32, device=device),
            "nxt": torch.zeros(16, dtype=torch.int32, device=device), "rids": None}

    def apply_events():
        for ev in script.pop_events():
            if ev[0] == "admit":
                pool.request_admit(ev[1], ev[2])
            else:
                pool.request_release(ev[1])

    bytes_log = []
    kv_tokens_log = []
    touched = {"mean": None}    # mean distinct experts per layer a step routes to (measured in the profile pass)

    def one_step(mode, want_logits=False):
        """mode 'chained': the fed-in tokens stay on the device; 'host': q4d_decode_step_host."""
        script.churn()
        apply_events()
        ids, toks, lens, bt = script.step_inputs()
        bytes_log.append(step_bytes(shape, lens, len(ids), touched["mean"]))
        kv_tokens_log.append(float(np.mean(lens)) + 1.0)
        if mode == "host":
            out, _ = q4d.decode_step_host(model, pool, ids, toks, bt, want_logits=want_logits)
            script.advance(out)
            bufs["rids"] = None
            return len(ids)
        rids = ids.tolist()
        if bufs["rids"] == rids:
            bufs["cur"], bufs["nxt"] = bufs["nxt"], bufs["cur"]      # previous outputs are this step's inputs
        else:
            # membership changed: survivors keep their previous output, new requests feed their first token
            prev = {r: i for i, r in enumerate(bufs["rids"] or [])}
            src = torch.tensor([prev.get(r, 0) for r in rids], dtype=torch.long, device=device)
            new = torch.tensor([r not in prev for r in rids], dtype=torch.bool, device=device)
            first = torch.from_numpy(toks).to(device)
            bufs["cur"][:len(rids)] = torch.where(new, first, bufs["nxt"][src])
        q4d.decode_step_chained(model, pool, ids, bufs["cur"], bt, bufs["nxt"])
        script.advance()
        bufs["rids"] = rids
        return len(ids)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    apply_events()
    for _ in range(args.warmup):
        one_step("chained")
    # ---- timed region 1: device-resident throughput ----
    visible = [v for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v]
    sampler = ClockSampler(visible[local_rank] if local_rank < len(visible) else local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier()
    launches0 = model.launch_count()
    bytes_log.clear()
    kv_tokens_log.clear()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    e0.record(stream)
    tokens = 0
    for _ in range(args.steps):
        tokens += one_step("chained")
    e1.record(stream)
    barrier()
    wall1 = time.time()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(wall0, wall1)
    launches = model.launch_count() - launches0
    timed_bytes = list(bytes_log)
    mean_kv_tokens = float(np.mean(kv_tokens_log))

    # host time to submit one step into an empty stream (if this approaches ms_per_step the host is the limit)
    submit = []
    for _ in range(4):
        torch.cuda.synchronize()
        t_s0 = time.perf_counter()
        one_step("chained")
        submit.append((time.perf_counter() - t_s0) * 1e3)
    torch.cuda.synchronize()
    host_enqueue_ms = float(np.median(submit))

    # ---- timed region 2: the same steps through the host-buffer entry point ----
    barrier()
    t_host0 = time.perf_counter()
    tokens_e2e = 0
    for _ in range(args.steps):
        tokens_e2e += one_step("host")
    torch.cuda.synchronize()
    ms_e2e = (time.perf_counter() - t_host0) * 1e3   # every step ends with a stream sync, so host time is device time
    barrier()
    h2d, d2h = model.step_io_bytes()
    # the same entry point with the logits copied back as well (n x vocab x 4 bytes per step), on fewer steps
    logit_steps = max(1, min(args.steps, 16))
    t_host0 = time.perf_counter()
    tokens_lg = 0
    for _ in range(logit_steps):
        tokens_lg += one_step("host", want_logits=True)
    torch.cuda.synchronize()
    ms_e2e_lg = (time.perf_counter() - t_host0) * 1e3
    h2d_lg, d2h_lg = model.step_io_bytes()

    # ---- the neighbouring rows of the path, on the same model: prompt processing and sampling ----
    def timed_ms(fn, reps=3):
        best = 1e30
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        return best

    extras = {}
    try:
        prompt = np.random.default_rng(seed + 5).integers(0, shape.vocab, size=512).astype(np.int32)
        pblocks = script.alloc.alloc(33)
        rid = [10 ** 9]

        def run_prefill(start):
            q4d.prefill(model, pool, rid[0], prompt, start, pblocks)
            pool.request_release(rid[0])
            rid[0] += 1

        t_full = timed_ms(lambda: run_prefill(0))
        t_hit = timed_ms(lambda: run_prefill(496))       # a 496-token prefix already cached: 16 tokens to process
        extras["prefill"] = {"prompt_tokens": 512, "ttft_ms": t_full, "tokens_per_s": 512 / (t_full * 1e-3),
                             "ttft_ms_with_496_cached": t_hit, "speedup_from_prefix_cache": t_full / t_hit,
                             "note": "q4d_prefill: sixteen tokens per pass over the weights (not a compute-bound "
                                     "kernel yet); the paper's Table 7 reports 245 ms -> 42 ms on its hardware"}
        script.alloc.release(pblocks)
        lg = torch.randn(n, shape.vocab, device=device)
        us = np.random.default_rng(seed + 6).uniform(0, 1, size=n).astype(np.float32)
        t_s = timed_ms(lambda: q4d.sample(lg, [0.8] * n, [50] * n, [0.95] * n, us), reps=5)
        extras["sampling"] = {"us_per_step": t_s * 1e3, "settings": "temperature 0.8, top-k 50, top-p 0.95",
                              "share_of_step": t_s / (ms / args.steps)}
    except Exception as ex:  # the headline numbers do not depend on these
        extras["error"] = repr(ex)

    # ---- per-launch timing (events around every launch) for the roofline of the dominant kernel ----
    fused = model.is_fused()
    model.profile_enable(True)
    if fused:
        model.timeline_enable(True)
    bytes_log.clear()
    touched_counts = []
    for _ in range(args.profile_steps):
        one_step("chained")
        if shape.n_experts:
            touched_counts.append(model.moe_touched_experts() / shape.n_layers)
    torch.cuda.synchronize()
    if touched_counts:
        touched["mean"] = float(np.mean(touched_counts))
    prof = model.profile_read()
    model.profile_enable(False)
    peak, peak_kind = peaks()
    if fused:
        # one persistent kernel runs the whole step: its algorithmic bytes are the step's
        step_ms, step_cnt = prof["fused_step"]
        per_launch = float(np.mean([b["total"] for b in bytes_log]))
        gbs = per_launch / (step_ms / step_cnt * 1e-3) / 1e9 if step_cnt else 0.0
        roofline = {"kernel": "fused_step_kernel", "bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s",
                    "frac": gbs / peak, "peak_kind": peak_kind, "traffic": None, "bytes_per_launch": per_launch,
                    "us_per_launch": step_ms / max(step_cnt, 1) * 1e3,
                    "timing": "CUDA events around each launch, profile pass right after the timed steps"}
        tl = model.timeline_read()      # phases of the last profiled step, from the kernel's own clock stamps
        model.timeline_enable(False)
        tl_total = sum(v[0] for v in tl.values()) or 1.0
        kernels = {k: {"us_per_step": v[0], "phases_per_step": v[1], "share": v[0] / tl_total} for k, v in tl.items()}
    else:
        # The dominant kernel is the one whose launches take the largest share of the step; the algorithmic bytes of a
        # launch are the packed tensor it streams (projections) or the cached K, V it reads (attention).
        from workload import shapes as shp
        H, d = shape.hidden, shape.head_dim
        kv_read_layer = float(np.mean([b["kv_read"] for b in bytes_log])) / shape.n_layers
        class_bytes = {"gemm_qkv": shp.q4_bytes(shape.qkv_out, H), "gemm_o": shp.q4_bytes(H, shape.n_q_heads * d),
                       "gemm_gate_up": shp.q4_bytes(2 * shape.mlp_inter, H) if shape.mlp_inter else 0,
                       "gemm_down": shp.q4_bytes(H, shape.mlp_inter) if shape.mlp_inter else 0,
                       "lm_head": shp.q4_bytes(shape.vocab, H) + n * shape.vocab * 4, "attention": kv_read_layer}
        if shape.n_experts:  # distinct experts per layer, counted from the routing of the profiled steps
            class_bytes["moe_gate_up"] = touched["mean"] * shp.q4_bytes(2 * shape.expert_inter, H)
            class_bytes["moe_down"] = touched["mean"] * shp.q4_bytes(H, shape.expert_inter)
        proj = "q4_umma_kernel" if os.environ.get("Q4D_GEMM_KERNEL") == "tcgen05" else "q4_span_kernel"
        head = "q4_umma_kernel" if os.environ.get("Q4D_GEMM_KERNEL") == "tcgen05" else "q4_round_kernel"
        class_kernel = {"gemm_qkv": proj, "gemm_o": proj, "gemm_gate_up": proj, "gemm_down": proj, "lm_head": head,
                        "attention": ("paged_attention_t_kernel" if shape.n_q_heads // shape.n_kv_heads <= 8
                                      else "paged_attention_kernel"), "moe_gate_up": "q4_gemm_kernel",
                        "moe_down": "q4_gemm_kernel", "rmsnorm": "rmsnorm_kernel", "embed": "embed_kernel",
                        "argmax": "argmax_finish_kernel", "moe_router": "moe_router_kernel"}
        # DRAM bytes per algorithmic byte from one `ncu --set full` capture of each kernel (see profiles/: the span kernel
        # on a gate/up-shaped projection alone, attention on the Llama-3.2-3B-shaped batch-16 case); traffic is
        # proportional to the bytes streamed, so it is scaled to this launch.
        traffic_ratio = {"q4_span_kernel": 1.005, "paged_attention_t_kernel": 1.037}
        total_prof_ms = sum(v[0] for v in prof.values())
        classes = {k: {"ms_per_step": v[0] / args.profile_steps, "launches_per_step": v[1] / args.profile_steps,
                       "share": v[0] / total_prof_ms, "kernel": class_kernel.get(k, k)} for k, v in prof.items() if v[1]}
        for k, v in classes.items():
            if k in class_bytes and prof[k][1]:
                v["GBps"] = class_bytes[k] / (prof[k][0] / prof[k][1] * 1e-3) / 1e9
        # one entry per kernel: its launches of every class added up
        kernels = {}
        for k, v in classes.items():
            e = kernels.setdefault(v["kernel"], {"ms_per_step": 0.0, "launches_per_step": 0.0, "share": 0.0,
                                                 "bytes_per_step": 0.0, "classes": []})
            e["ms_per_step"] += v["ms_per_step"]
            e["launches_per_step"] += v["launches_per_step"]
            e["share"] += v["share"]
            e["bytes_per_step"] += class_bytes.get(k, 0.0) * v["launches_per_step"]
            e["classes"].append(k)
        for e in kernels.values():
            e["GBps"] = e["bytes_per_step"] / (e["ms_per_step"] * 1e-3) / 1e9 if e["bytes_per_step"] else None
        top = max((k for k in kernels if kernels[k]["bytes_per_step"]), key=lambda k: kernels[k]["share"])
        te = kernels[top]
        per_launch_bytes = te["bytes_per_step"] / te["launches_per_step"]
        gbs = te["GBps"]
        roofline = {"kernel": top, "bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                    "peak_kind": peak_kind, "share_of_step": te["share"],
                    "traffic": per_launch_bytes * traffic_ratio[top] if top in traffic_ratio else None,
                    "bytes_per_launch": per_launch_bytes,
                    "us_per_launch": te["ms_per_step"] / te["launches_per_step"] * 1e3,
                    "launches_per_step": te["launches_per_step"],
                    "classes": {k: {"GBps": classes[k].get("GBps"), "frac": classes[k].get("GBps", 0.0) / peak,
                                    "us_per_launch": classes[k]["ms_per_step"] / classes[k]["launches_per_step"] * 1e3,
                                    "share_of_step": classes[k]["share"]} for k in te["classes"]},
                    "timing": "CUDA events around each launch (a pass of --profile-steps steps right after the timed "
                              "steps); achieved = bytes of all launches of the kernel / their summed time"}
        kernels["by_class"] = classes

    # ---- max over ranks, aggregate ----
    ms, ms_e2e, tokens, tokens_e2e, launches = aggregate_ranks(dist, device, ms, ms_e2e, tokens, tokens_e2e, launches)

    # bytes of the timed steps (mixture of experts: with the routed-expert count measured in the profile pass)
    from workload import shapes as shp2
    mean_bytes = {k: float(np.mean([b[k] for b in timed_bytes])) for k in timed_bytes[0]}
    if shape.n_experts:
        w_meas = float(shp2.weight_bytes(shape, touched["mean"]))
        mean_bytes["total"] += w_meas - mean_bytes["weights"]
        mean_bytes["weights"] = w_meas
        config["experts"] = (f"{shape.n_experts} experts, top-{shape.top_k}; weight bytes count the distinct experts "
                             f"the steps routed to (q4d_moe_touched_experts: {touched['mean']:.1f} per layer, mean over "
                             f"the {args.profile_steps} profiled steps)")
    config["workload"] += f"; mean cached tokens per request over the {args.steps} timed steps: {mean_kv_tokens:.0f}"
    config["kv_mix"] = ("not stationary: departing requests are replaced by 512-token ones, so the mean KV length "
                        "falls as steps go by; compare runs of equal --steps only") if churn else "fixed set of requests"

    value = tokens / (ms * 1e-3)
    step_gbs = mean_bytes["total"] / (ms / args.steps * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config,
        "step_bytes": mean_bytes,
        "step_hbm": {"achieved_GBps": step_gbs, "frac_of_measured_copy_peak": step_gbs / peak,
                     "frac_of_8TBps_nominal": step_gbs / 8000.0, "peak_kind": peak_kind},
        "roofline": roofline,
        "kernels": kernels,
        "e2e": {"value": tokens_e2e / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps,
                "returns": "next tokens only (the logits stay on the device)"},
        "e2e_with_logits": {"value": tokens_lg / (ms_e2e_lg * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": h2d_lg,
                            "d2h_bytes_per_step": d2h_lg, "ms_per_step": ms_e2e_lg / logit_steps, "steps": logit_steps,
                            "returns": "next tokens and the fp32 logits of every request"},
        "gpu_launches": launches,
        "clocks": clocks,
        "host_submit_ms_per_step": host_enqueue_ms,
        "extras": extras,
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # The oracle on whole steps of this workload; its result for the step is also the parity check of the run:
        # the GPU takes the same step (same tokens, same KV) and the logits and greedy tokens are compared.
        ids, toks, lens, bt = script.step_inputs()
        t_step, timed, desc, cores, (o_next, o_logits) = oracle_steps(shape, weights, pool_t, lens, toks, bt, 3,
                                                                      args.oracle_budget)
        out["cpu_baseline"] = {"value": len(ids) / t_step, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                               "sample": desc}
        g_next = torch.zeros(len(ids), dtype=torch.int32, device=device)
        g_logits = torch.zeros(len(ids), shape.vocab, dtype=torch.float32, device=device)
        q4d.decode_step(model, pool, ids, toks, bt, g_next, g_logits)
        torch.cuda.synchronize()
        gl, ol = g_logits.cpu().numpy().astype(np.float64), o_logits.astype(np.float64)
        rms = np.sqrt((ol ** 2).mean(-1))
        out["parity"] = {"kind": "one whole step of this workload against the oracle, free-running through all "
                                 f"{shape.n_layers} layers (bf16 rounding differences compound with depth; the "
                                 "teacher-forced per-layer and head checks are in tests/)",
                         "max_dlogit_over_rms": float((np.abs(gl - ol).max(-1) / rms).max()),
                         "rms_dlogit_over_rms": float((np.sqrt(((gl - ol) ** 2).mean(-1)) / rms).max()),
                         "greedy_tokens_equal": int((g_next.cpu().numpy() == o_next).sum()), "of": int(len(ids))}
    if rank == 0:
        print(json.dumps(out))
    pool.close()
    model.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
