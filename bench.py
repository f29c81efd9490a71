"""Decode-throughput benchmark of the q4decode library (one JSON line on stdout).

A step is one decode step of the whole batch (every kernel of the path).  The default workload is the
Qwen3-8B-shaped model at batch 16 with KV lengths drawn log-uniformly from [256, 8192] and four requests
leaving and four joining (512 prefilled tokens) every 32 steps; `--workload` selects the other shapes.

  value      tokens/s with everything resident in HBM (tokens chained on the device, no host sync)
  e2e        tokens/s through q4d_decode_step_host: host inputs, host outputs, a sync per step
  roofline   the dominant kernel (the launch class with the largest share of the step: a 4-bit projection or the
             paged attention) timed with CUDA events around each of its launches
  cpu_baseline  the CPU oracle on a bounded sample of the same step, on the host cores

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


def step_bytes(shape, lens, n):
    """Algorithmic bytes of one step: packed weights + scales + biases, KV read and written, logits, embedding rows."""
    from workload import shapes
    # mixture of experts: the experts a step touches depend on the routing; the expectation under uniform routing
    # (E * (1 - (1 - k/E)^n) distinct experts per layer) stands in for the count, which the library does not export
    touched = None
    if shape.n_experts:
        touched = shape.n_experts * (1.0 - (1.0 - shape.top_k / shape.n_experts) ** n)
    w = shapes.weight_bytes(shape, touched)
    per_tok_layer = 2 * shape.n_kv_heads * shape.head_dim * 2
    kv_read = int(sum(int(l) + 1 for l in lens)) * per_tok_layer * shape.n_layers
    kv_write = n * per_tok_layer * shape.n_layers
    logits = n * shape.vocab * 4
    embed_rows = n * shapes.q4_bytes(1, shape.hidden)
    return {"weights": w, "kv_read": kv_read, "kv_write": kv_write, "logits": logits, "embed": embed_rows,
            "total": w + kv_read + kv_write + logits + embed_rows}


def oracle_sample(shape, weights, pool_t, lens, toks, bt, budget_layers):
    """Times the oracle on a bounded sample of one step: the embedding + final norm + LM head alone, then the same
    with the first `budget_layers` layers; the full-step time is extrapolated by layer count.  Returns
    (seconds per full step, description, threads)."""
    from oracle import q4d_oracle as orc
    Ls = max(1, min(budget_layers, shape.n_layers))
    sub = dict(weights)
    sub["layers"] = weights["layers"][:Ls]
    om = orc.OracleModel(shape, sub)
    host_pool = orc.to_np(pool_t[:Ls]).copy()
    t0 = time.perf_counter()
    om.decode_step(host_pool, 16, lens, toks, bt, layer_limit=0, want_logits=False)
    t_head = time.perf_counter() - t0
    t0 = time.perf_counter()
    om.decode_step(host_pool, 16, lens, toks, bt, layer_limit=Ls, want_logits=False)
    t_ls = time.perf_counter() - t0
    full = t_head + (t_ls - t_head) * shape.n_layers / Ls
    desc = (f"one step of this workload (n={len(lens)}): LM head timed alone ({t_head:.2f} s) and with the first {Ls} "
            f"of {shape.n_layers} layers ({t_ls:.2f} s); per-step time extrapolated by layer count")
    return full, desc, orc.num_threads()


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3-8b-b16", choices=sorted(WORKLOADS))
    ap.add_argument("--profile-steps", type=int, default=8)
    ap.add_argument("--oracle-layers", type=int, default=4, help="layers in the CPU-baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()

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
    total_steps = args.warmup + 2 * args.steps + args.profile_steps + 8
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
        # The reference arm is the CPU oracle: every "step" is the same bounded sample, extrapolated to a full step.
        ids, toks, lens, bt = script.step_inputs()
        times, cores, desc = [], 0, ""
        for i in range(args.warmup + args.steps):
            full, desc, cores = oracle_sample(shape, weights, pool_t, lens, toks, bt, args.oracle_layers)
            if i >= min(args.warmup, 1):
                times.append(full)
            if sum(times) > 150 or len(times) >= args.steps:
                break
        t = float(np.mean(times))
        v = n / t
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s", "n_gpus": 0,
                          "steps": len(times), "warmup": min(args.warmup, 1), "ms_per_step": t * 1e3,
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

    def one_step(mode):
        """mode 'chained': the fed-in tokens stay on the device; 'host': q4d_decode_step_host."""
        script.churn()
        apply_events()
        ids, toks, lens, bt = script.step_inputs()
        bytes_log.append(step_bytes(shape, lens, len(ids)))
        if mode == "host":
            out, _ = q4d.decode_step_host(model, pool, ids, toks, bt)
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
    mean_bytes = {k: float(np.mean([b[k] for b in bytes_log])) for k in bytes_log[0]}

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

    # ---- per-launch timing (events around every launch) for the roofline of the dominant kernel ----
    fused = model.is_fused()
    model.profile_enable(True)
    if fused:
        model.timeline_enable(True)
    bytes_log.clear()
    for _ in range(args.profile_steps):
        one_step("chained")
    torch.cuda.synchronize()
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
        # The dominant kernel is the launch class with the largest share of the step; its algorithmic bytes per
        # launch are the packed tensor it streams (projections) or the cached K, V it reads (attention).
        from workload import shapes as shp
        H, d = shape.hidden, shape.head_dim
        kv_read_layer = float(np.mean([b["kv_read"] for b in bytes_log])) / shape.n_layers
        class_bytes = {"gemm_qkv": shp.q4_bytes(shape.qkv_out, H), "gemm_o": shp.q4_bytes(H, shape.n_q_heads * d),
                       "gemm_gate_up": shp.q4_bytes(2 * shape.mlp_inter, H) if shape.mlp_inter else 0,
                       "gemm_down": shp.q4_bytes(H, shape.mlp_inter) if shape.mlp_inter else 0,
                       "lm_head": shp.q4_bytes(shape.vocab, H) + n * shape.vocab * 4, "attention": kv_read_layer}
        if shape.n_experts:  # expected distinct experts per layer (see step_bytes)
            touched = shape.n_experts * (1.0 - (1.0 - shape.top_k / shape.n_experts) ** n)
            class_bytes["moe_gate_up"] = touched * shp.q4_bytes(2 * shape.expert_inter, H)
            class_bytes["moe_down"] = touched * shp.q4_bytes(H, shape.expert_inter)
        class_kernel = {"attention": "paged_attention_kernel", "lm_head": "q4_round_kernel", "moe_gate_up": "q4_gemm_kernel", "moe_down": "q4_gemm_kernel"}
        # DRAM bytes per algorithmic byte from one `ncu --set full` capture of each kernel on the Llama-3.2-3B-shaped
        # batch-16 case (see profiles/); traffic is proportional to the bytes streamed, so it is scaled to this launch.
        traffic_ratio = {"gemm_gate_up": 1.005, "attention": 1.032}
        total_prof_ms = sum(v[0] for v in prof.values())
        kernels = {k: {"ms_per_step": v[0] / args.profile_steps, "launches_per_step": v[1] / args.profile_steps,
                       "share": v[0] / total_prof_ms} for k, v in prof.items() if v[1]}
        for k, v in kernels.items():
            if k in class_bytes and prof[k][1]:
                v["GBps"] = class_bytes[k] / (prof[k][0] / prof[k][1] * 1e-3) / 1e9
        top = max((k for k in kernels if k in class_bytes), key=lambda k: kernels[k]["share"])
        top_ms, top_cnt = prof[top]
        gbs = class_bytes[top] / (top_ms / top_cnt * 1e-3) / 1e9
        roofline = {"kernel": class_kernel.get(top, "q4_span_kernel") + " (" + top + ")", "bound": "hbm", "achieved": gbs,
                    "peak": peak, "unit": "GB/s", "frac": gbs / peak, "peak_kind": peak_kind,
                    "traffic": class_bytes[top] * traffic_ratio[top] if top in traffic_ratio else None,
                    "bytes_per_launch": float(class_bytes[top]), "us_per_launch": top_ms / top_cnt * 1e3,
                    "timing": "CUDA events around each launch, profile pass right after the timed steps"}

    # ---- max over ranks, aggregate ----
    ms, ms_e2e, tokens, tokens_e2e, launches = aggregate_ranks(dist, device, ms, ms_e2e, tokens, tokens_e2e, launches)

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
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": launches,
        "clocks": clocks,
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ids, toks, lens, bt = script.step_inputs()
        full, desc, cores = oracle_sample(shape, weights, pool_t, lens, toks, bt, args.oracle_layers)
        out["cpu_baseline"] = {"value": len(ids) / full, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                               "sample": desc}
    if rank == 0:
        print(json.dumps(out))
    pool.close()
    model.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
