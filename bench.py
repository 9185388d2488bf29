"""Benchmark of one PosS speculative round on the Llama-3-8B-shaped drafter workload (config c2).

A step = the whole hot path once: poss_draft_round (6 specialist steps, width 10, 60 kept tokens,
prefix 1024) + the tree-masked target pass over the 61 tree rows (32 Llama-3-8B-shaped layers, final
norm, LM-head argmax) + the greedy accept walk + KV compaction.  Drafter weights and inputs come from
the seeded host generator (poss_synth); the 14 GB of target layers are drawn on the device from a
seeded generator (same recipe, N(0, 0.02) bf16) so that the default run stays within minutes.
With --no-target the step's verification side is the stand-alone stages instead (61-row attention at
target geometry, argmax over given logits, accept walk).  One JSON line on stdout.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config c2]
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

METRIC = "poss_draft_round_us_60tok_depth6"
# DRAM bytes (read + written) of one LM-head launch of k_gemm_tc at the Llama-3-8B shape, from the ncu capture whose
# summary is the named file (None once the kernel has changed since the capture)
TRAFFIC = {"bytes": 1050830000 + 3845888, "workloads": ("c2", "c4", "c5"),
           "source": "profiles/k_gemm_tc_c2_m10_gateup_down_lmhead.md, third captured launch (-s 9 -c 3: the LM head)"}


def algorithmic_bytes(cfg):
    """Bytes one draft round must move (bf16 weights of every matrix product + the active prefix KV)."""
    H, F, V = cfg.hidden, cfg.ffn, cfg.vocab
    qd, kd = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    per_step = 2 * (2 * H * H + H * (qd + 2 * kd) + qd * H + 3 * H * F + V * H) + 2 * 2 * kd * cfg.prefix
    return per_step * cfg.depth, 2 * V * H


class ClockSampler:
    """One `nvidia-smi -lms` process for the whole measurement; samples are stamped on arrival and the summary
    keeps those that fell inside the timed regions."""
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
        "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, gpu_id: str, period_ms: int = 20):
        self.rows, self.windows, self.proc = [], [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", str(period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            return
        self.t = threading.Thread(target=self._read, daemon=True)
        self.t.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.strip().split(",")]))

    def window(self, t0: float, t1: float):
        self.windows.append((t0, t1))

    def close(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        inside = [r for t, r in self.rows if len(r) >= 7 and any(a <= t <= b for a, b in self.windows)]
        num = lambda x: x.replace(".", "", 1).isdigit()
        sm = [float(r[0]) for r in inside if num(r[0])]
        mx = [float(r[1]) for r in inside if num(r[1])]
        pw = [float(r[2]) for r in inside if num(r[2])]
        reasons = []
        for name, col in (("hw_slowdown", 3), ("hw_thermal_slowdown", 4), ("sw_thermal_slowdown", 5), ("sw_power_cap", 6)):
            if any(r[col].lower().startswith("active") for r in inside):
                reasons.append(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "reasons": reasons, "samples": len(sm)}


def replica_seed(rank: int) -> int:
    """Replicas only: every rank runs its own request, drawn from its own seed."""
    return 1 + rank


def slowest_rank(times_ms, world: int, device):
    """Per-step times of this rank -> the job's: the maximum over ranks (every replica must have finished)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def rounds_per_second(world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank completes one round per step."""
    return world * 1e3 / ms_per_step


def workload_name(cfg) -> str:
    """The drafter workload, worded identically by both arms."""
    shape = "Llama-3-8B" if cfg.hidden == 4096 else "Llama-2-13B" if cfg.hidden == 5120 else "test"
    return (f"{cfg.name}: drafter H={cfg.hidden} F={cfg.ffn} V={cfg.vocab} ({shape}-shaped), {cfg.S} specialists x {cfg.n} "
            f"positions, depth {cfg.depth}, top-k {cfg.topk}, {cfg.total} tokens, prefix {cfg.prefix}")


def chain_spans(records):
    """Timeline records [(kernel name, ns)] in time order -> {phase: {kernel: [launches, summed span in us]}}.
    A record is the instant a launch's wait for its predecessor returned; the span of a launch inside the chain is
    the time to the next record.  Phases: a draft round runs from its first gather_x to its rerank, a target pass
    from embed_rows to the accept walk; the last record of a phase has no successor inside it and is left out."""
    out = {"draft": {}, "target": {}}
    phase = None
    for i, (name, t) in enumerate(records):
        if name == "gather_x" and phase != "draft":
            phase = "draft"
        elif name == "embed_rows":
            phase = "target"
        if phase is None or i + 1 >= len(records):
            continue
        nxt_name, nxt_t = records[i + 1]
        ends = (phase == "draft" and name == "rerank") or (phase == "target" and name == "accept_walk")
        if not ends:
            cell = out[phase].setdefault(name, [0, 0.0])
            cell[0] += 1
            cell[1] += (nxt_t - t) / 1e3
        if ends:
            phase = None
    return out


def run_batched(args, cfg):
    """--batch B: the draft round for B independent sequences in one call (poss_draft_round_batched), timed like
    the single round; one JSON line with the batched round's time and the sequences drafted per second."""
    import torch
    import poss_synth as ps
    from paper_2506_03566_b200 import Poss, make_config, to_device
    from paper_2506_03566_b200 import build as pbuild
    pbuild.build()
    torch.cuda.set_device(0)
    B = args.batch
    seed = replica_seed(0)
    w = ps.make_weights(cfg, seed, alias_specialists=args.alias_specialists)
    cap = cfg.prefix + 8 + cfg.tree_slots
    P = Poss(make_config(cfg, cap, 0, max_batch=B), w)
    del w
    kvs = [to_device(ps.make_draft_kv(cfg, seed + 100 * b, cap)) for b in range(B)]
    ins = [ps.make_round_inputs(cfg, seed + 100 * b, 1) for b in range(B)]
    tok = torch.from_numpy(np.concatenate([t for t, _ in ins])).cuda()
    feat = to_device(np.concatenate([f for _, f in ins], axis=0))
    pl, nn = [cfg.prefix] * B, [1] * B
    out = P.poss_draft_round_batched(kvs, pl, tok, feat, nn, cfg.depth, cfg.topk, cfg.total)
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        P.poss_draft_round_batched(kvs, pl, tok, feat, nn, cfg.depth, cfg.topk, cfg.total, out=out)
    torch.cuda.synchronize()
    assert P.poss_last_status() == 0
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(0).uuid)
    except Exception:
        gpu_id = "0"
    clocks = ClockSampler(gpu_id)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = P.poss_launch_count()
    t_a = time.perf_counter()
    e0.record()
    for _ in range(args.steps):
        P.poss_draft_round_batched(kvs, pl, tok, feat, nn, cfg.depth, cfg.topk, cfg.total, out=out)
    e1.record()
    torch.cuda.synchronize()
    clocks.window(t_a, time.perf_counter())
    clocks.close()
    ms = e0.elapsed_time(e1) / args.steps
    P.poss_profile(3)
    for _ in range(min(args.steps, 5)):
        P.poss_draft_round_batched(kvs, pl, tok, feat, nn, cfg.depth, cfg.topk, cfg.total, out=out)
    chain = chain_spans(P.poss_timeline_read())["draft"]
    P.poss_profile(0)
    try:
        hbm_peak, which = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["hbm_gbs"]), "measured"
    except Exception:
        hbm_peak, which = 6650.0, "fallback"
    round_bytes, _ = algorithmic_bytes(cfg)
    # tensor work of the round: 2 x rows x weights per step (rows = B x K current rows; pending rows left out)
    H, F, V = cfg.hidden, cfg.ffn, cfg.vocab
    qd, kd = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    w_elems = 2 * H * H + H * (qd + 2 * kd) + qd * H + 3 * H * F + V * H
    flops = sum(2.0 * B * (1 if i == 0 else cfg.topk) * w_elems for i in range(cfg.depth))
    line = {"metric": METRIC, "value": ms * 1e3, "unit": "us", "n_gpus": 1, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": workload_name(cfg), "batch": B,
                       "step": f"one batched draft round: {B} independent sequences drafted in one call",
                       "l2": "inputs larger than L2 (1.56 GB of weights per specialist step)"},
            "batch": B, "us_per_sequence": ms * 1e3 / B, "sequences_per_s": B * 1e3 / ms,
            "weight_stream_gbs": round_bytes / (ms * 1e-3) / 1e9,
            "weight_stream_frac_of_hbm_peak": round_bytes / (ms * 1e-3) / 1e9 / hbm_peak, "peak_source": which,
            "tensor_tflops": flops / (ms * 1e-3) / 1e12,
            "gpu_launches": int((P.poss_launch_count() - launches0) // args.steps),
            "chain_us_per_launch": {n: round(c[1] / c[0], 2) for n, c in sorted(chain.items())},
            "clocks": clocks.summary()}
    print(json.dumps(line))


def run_reference(args, cfg):
    """The oracle, as it stands, on the host cores: one full draft round per step."""
    import poss_synth as ps
    from oracle import poss_oracle as po
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = ps.make_weights(cfg, 1)
    cap = cfg.prefix + 1 + cfg.tree_slots
    kv = ps.make_draft_kv(cfg, 1, cap)
    tok, feat = ps.make_round_inputs(cfg, 1, 1)
    num = po.Num(np.float32, "bf16")
    kvw = po.widen(kv, num.dtype)
    steps, warm = max(1, min(args.steps, 3)), min(args.warmup, 1)
    for _ in range(warm):
        po.draft_round(cfg, w, kvw.copy(), cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total, num)
    t0 = time.perf_counter()
    for _ in range(steps):
        po.draft_round(cfg, w, kvw.copy(), cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total, num)
    dt = (time.perf_counter() - t0) / steps
    us = dt * 1e6
    cores = len(os.sched_getaffinity(0))
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": "us", "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "step": "one draft round (the metric's quantity)"},
            "cpu_baseline": {"value": us, "unit": "us", "cores": cores, "kind": "oracle",
                             "sample": "one full draft round (numpy fp32, bf16 rounding contract); verify stages not included"},
            "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--config", default="c2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--depth", type=int, help="override the workload's draft depth L")
    ap.add_argument("--total", type=int, help="override the workload's kept draft tokens T")
    ap.add_argument("--specialists", type=int, help="override the number of position specialists S")
    ap.add_argument("--positions", type=int, help="override the positions per specialist n (PosS-n)")
    ap.add_argument("--batch", type=int, default=1,
                    help="B > 1: time poss_draft_round_batched for B independent sequences (draft round only, 1 GPU)")
    ap.add_argument("--no-target", action="store_true", help="verification side = stand-alone stages, no target layers")
    ap.add_argument("--alias-specialists", action="store_true",
                    help="profiler captures only: all specialists share one weight set, so the process holds "
                         "about 3 GB instead of 10 GB; the launch chain and every launch's traffic are unchanged "
                         "(one step still streams 1.56 GB, far more than L2)")
    ap.add_argument("--target-layers", type=int,
                    help="layers of the target pass (default 32, the workload; 0 with --alias-specialists).  Fewer "
                         "layers keep a profiler capture of the target-pass kernels small: every layer launches the "
                         "same kernels on the same shapes")
    args = ap.parse_args()

    import poss_synth as ps
    cfg = ps.CONFIGS[args.config]
    over = {k: v for k, v in (("depth", args.depth), ("total", args.total), ("S", args.specialists), ("n", args.positions))
            if v is not None}
    if over:
        cfg = cfg.replace(**over)
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if args.batch > 1:
        run_batched(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2506_03566_b200 import Poss, make_config, to_device
    from paper_2506_03566_b200 import build as pbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        pbuild.build()
    if world > 1:
        dist.barrier()
    warmup = max(args.warmup, 3)

    # ---------------- inputs: seeded, resident in HBM before timing
    seed = replica_seed(rank)
    n_layers = args.target_layers if args.target_layers is not None else (0 if args.alias_specialists else 32)
    with_target = not args.no_target and n_layers > 0
    if not with_target:
        n_layers = 0
    w = ps.make_weights(cfg, seed, alias_specialists=args.alias_specialists)
    rows = cfg.total + 1
    cap = cfg.prefix + 8 + cfg.tree_slots
    tcap = cfg.prefix + rows
    if with_target:
        gen = torch.Generator(device="cuda").manual_seed(1000 + seed)
        H, F = cfg.hidden, cfg.ffn
        qd, kd = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim

        def dev_normal(*shape, std=0.02):
            return (torch.randn(*shape, device="cuda", generator=gen) * std).to(torch.bfloat16)

        def dev_gain():
            return (1.0 + 0.1 * torch.randn(H, device="cuda", generator=gen)).to(torch.bfloat16)

        w["target"] = [{"norm_in": dev_gain(), "wq": dev_normal(qd, H), "wk": dev_normal(kd, H), "wv": dev_normal(kd, H),
                        "wo": dev_normal(H, qd), "norm_post": dev_gain(), "w_gate": dev_normal(F, H),
                        "w_up": dev_normal(F, H), "w_down": dev_normal(H, F)} for _ in range(n_layers)]
        w["final_norm"] = dev_gain()
    P = Poss(make_config(cfg.replace(n_target_layers=n_layers), cap, tcap), w)
    dkv = to_device(ps.make_draft_kv(cfg, seed, cap))
    tok_h, feat_h = ps.make_round_inputs(cfg, seed, 1)
    tok_pin = torch.from_numpy(tok_h).pin_memory()
    feat_pin = torch.from_numpy(feat_h.view(np.int16)).pin_memory()
    tok_d = tok_pin.cuda()
    feat_d = feat_pin.cuda().view(torch.bfloat16)
    scale = 1.0 / float(np.sqrt(cfg.head_dim))
    out = P.poss_draft_round(dkv, cfg.prefix, tok_d, feat_d, cfg.depth, cfg.topk, cfg.total)
    if with_target:
        # target cache: prefix keys / values N(0, 1), tree rows appended by the pass itself
        tkv_t = P.new_target_kv()
        tkv_t[:, :, :, :cfg.prefix, :] = torch.randn(n_layers, 2, cfg.n_kv_heads, cfg.prefix, cfg.head_dim, device="cuda",
                                                     generator=gen).to(torch.bfloat16)

        def step(tok, feat):
            tree = P.poss_draft_round(dkv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total, out=out)
            tf, targ, _ = P.poss_target_forward(tkv_t, cfg.prefix, tree["tokens"], tree["depth"], tree["anc_mask"], rows)
            va = P.poss_verify_accept(None, targ, tf, tree["tokens"], tree["parents"], rows)
            P.poss_kv_compact(tkv_t, cfg.prefix, va["path"], va["n_accepted"])
            return va
    else:
        # stand-alone verification stages: target-geometry KV with the tree rows' keys behind the prefix
        q_h, tkv_h = ps.make_attention_case(seed, rows, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.prefix, tcap, "bf16")
        q_d, tkv_d = to_device(q_h), to_device(tkv_h)
        logits_d = to_device(ps.normal(seed, "target_logits", (rows, cfg.vocab), 1.0, "bf16"))
        tfeat_d = to_device(ps.normal(seed, "target_features", (rows, cfg.hidden), 1.0, "bf16"))
        attn_out = torch.empty_like(q_d)

        def step(tok, feat):
            tree = P.poss_draft_round(dkv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total, out=out)
            P.poss_tree_attention(q_d, tkv_d, cfg.prefix, tree["anc_mask"], scale, out=attn_out)
            return P.poss_verify_accept(logits_d, None, tfeat_d, tree["tokens"], tree["parents"], rows)
    del w

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(warmup):
        step(tok_d, feat_d)
    sync_all()
    assert P.poss_last_status() == 0

    # ---------------- timed region 1: inputs resident in HBM
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    P.poss_profile(1)
    launches0 = P.poss_launch_count()
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        gpu_id = str(local)
    clocks = ClockSampler(gpu_id)
    time.sleep(0.3)                       # let the sampler come up before the timed region
    sync_all()
    t_a = time.perf_counter()
    ev[0].record()
    for _ in range(args.steps):
        step(tok_d, feat_d)
    ev[1].record()
    sync_all()
    clocks.window(t_a, time.perf_counter())
    ms = ev[0].elapsed_time(ev[1]) / args.steps
    launches = (P.poss_launch_count() - launches0) // args.steps
    n_lm, lm_ms = P.poss_profile_read()["lm_head"]
    P.poss_profile(0)

    # draft round alone (the metric's own quantity)
    sync_all()
    t_a = time.perf_counter()
    ev[2].record()
    for _ in range(args.steps):
        P.poss_draft_round(dkv, cfg.prefix, tok_d, feat_d, cfg.depth, cfg.topk, cfg.total, out=out)
    ev[3].record()
    sync_all()
    clocks.window(t_a, time.perf_counter())
    clocks.close()
    draft_ms = ev[2].elapsed_time(ev[3]) / args.steps

    # spread of single rounds: one event pair per round, in a loop of its own (the figures above stay averages
    # over back-to-back rounds without events in between)
    def spread(fn, n):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
        evs[0].record()
        for i in range(n):
            fn()
            evs[i + 1].record()
        torch.cuda.synchronize()
        t = sorted(evs[i].elapsed_time(evs[i + 1]) * 1e3 for i in range(n))
        return {"p10": t[int(0.1 * (n - 1))], "p50": t[(n - 1) // 2], "p90": t[int(0.9 * (n - 1) + 0.5)], "rounds": n}
    n_spread = max(5, min(args.steps, 30))
    spread_draft = spread(lambda: P.poss_draft_round(dkv, cfg.prefix, tok_d, feat_d, cfg.depth, cfg.topk, cfg.total, out=out),
                          n_spread)
    spread_step = spread(lambda: step(tok_d, feat_d), n_spread)
    sync_all()

    # every stage kind of the draft steps in isolation (events around each stage cut the launch overlap, so
    # this loop is slower than the round above and only feeds the per-kernel table)
    P.poss_profile(2)
    for _ in range(min(args.steps, 10)):
        P.poss_draft_round(dkv, cfg.prefix, tok_d, feat_d, cfg.depth, cfg.topk, cfg.total, out=out)
    per_kind = P.poss_profile_read()
    P.poss_profile(0)
    sync_all()

    # the same stages INSIDE the chain of dependent launches: every launch records the device time at which its wait
    # for its predecessor returned; a launch's span is the time to the next record (overlap included, nothing cut)
    P.poss_profile(3)
    n_chain = min(args.steps, 10)
    for _ in range(n_chain):
        step(tok_d, feat_d)
    chain = chain_spans(P.poss_timeline_read())
    P.poss_profile(0)
    sync_all()

    # ---------------- timed region 2: end to end through the C ABI with host buffers (host-timed)
    # (a) the metric's own quantity: pinned-host inputs -> device, draft round, tree back to pinned host
    res_host = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in out.items()}
    acc_host = torch.empty(2, dtype=torch.int32).pin_memory()
    h2d = tok_pin.numel() * 4 + feat_pin.numel() * 2
    d2h = sum(v.numel() * v.element_size() for v in res_host.values())
    sync_all()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        tok = tok_pin.cuda(non_blocking=True)
        feat = feat_pin.cuda(non_blocking=True).view(torch.bfloat16)
        P.poss_draft_round(dkv, cfg.prefix, tok, feat, cfg.depth, cfg.topk, cfg.total, out=out)
        for k, v in res_host.items():
            v.copy_(out[k], non_blocking=True)
        torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / args.steps
    # (b) the whole round the same way: accepted length and bonus token read back as well
    sync_all()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        tok = tok_pin.cuda(non_blocking=True)
        feat = feat_pin.cuda(non_blocking=True).view(torch.bfloat16)
        va = step(tok, feat)
        for k, v in res_host.items():
            v.copy_(out[k], non_blocking=True)
        acc_host[0:1].copy_(va["n_accepted"], non_blocking=True)
        acc_host[1:2].copy_(va["bonus"], non_blocking=True)
        torch.cuda.synchronize()
    e2e_round_ms = (time.perf_counter() - t0) * 1e3 / args.steps
    sync_all()

    ms, draft_ms, e2e_ms, e2e_round_ms = slowest_rank([ms, draft_ms, e2e_ms, e2e_round_ms], world, "cuda")

    if rank == 0:
        peaks, which = None, "fallback"
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
            which = "measured"
        except Exception:
            pass
        hbm_peak = float(peaks["hbm_gbs"]) if peaks else 6650.0
        round_bytes, lm_bytes = algorithmic_bytes(cfg)
        lm_dur = lm_ms / max(n_lm, 1)
        achieved = lm_bytes / (lm_dur * 1e-3) / 1e9 if n_lm else None
        line = {
            "metric": METRIC, "value": draft_ms * 1e3, "unit": "us", "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg),
                       "step": "draft round (the metric's quantity) + " +
                               (f"{rows}-row tree-masked pass of a {n_layers}-layer target of the same shape + accept walk + KV compaction"
                                if with_target else f"{rows}-row verification attention + logits argmax + accept walk"),
                       "l2": "inputs larger than L2 (1.56 GB of weights per specialist step)",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "stages_us": {"draft_round": draft_ms * 1e3, "whole_step": ms * 1e3,
                          "verify_round": max(ms - draft_ms, 0.0) * 1e3},
            "spread_us": {"draft_round": spread_draft, "whole_step": spread_step},
            "rounds_per_s": rounds_per_second(world, ms),
            "draft_round_gbs": round_bytes / (draft_ms * 1e-3) / 1e9,
            "draft_round_frac_of_hbm_peak": round_bytes / (draft_ms * 1e-3) / 1e9 / hbm_peak,
            "e2e": {"value": e2e_ms * 1e3, "unit": "us", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "what": "draft round incl. pinned-host input copy and read-back of the tree, host-timed",
                    "whole_round_us": e2e_round_ms * 1e3},
            "gpu_launches": int(launches),
            "clocks": clocks.summary(),
            "roofline": {"bound": "hbm", "kernel": "k_gemm_tc on the LM head (V x H bf16)", "achieved": achieved,
                         "peak": hbm_peak, "peak_source": which, "unit": "GB/s",
                         "frac": achieved / hbm_peak if achieved else None,
                         # dram__bytes_read.sum + dram__bytes_write.sum of one LM-head launch, from the ncu capture
                         # summarised in profiles/k_gemm_tc_c2_m10_gateup_down_lmhead.md (c2 shapes only)
                         "traffic": TRAFFIC["bytes"] if cfg.name in TRAFFIC["workloads"] else None,
                         "traffic_source": TRAFFIC["source"] if cfg.name in TRAFFIC["workloads"] else None,
                         "launches_timed": n_lm, "avg_launch_us": lm_dur * 1e3,
                         "algorithmic_bytes_per_launch": lm_bytes},
        }
        H_, F_, V_ = cfg.hidden, cfg.ffn, cfg.vocab
        qd_, kd_ = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
        avg_keys = cfg.prefix + 1 + cfg.topk * (cfg.depth - 1) / 2.0
        kind_bytes = {"fc": 2 * 2 * H_ * H_, "qkv": 2 * H_ * (qd_ + 2 * kd_), "attention": 2 * 2 * kd_ * avg_keys,
                      "o": 2 * qd_ * H_, "gate_up": 2 * 2 * F_ * H_, "down": 2 * F_ * H_, "lm_head": 2 * V_ * H_}
        line["kernels"] = {
            k: {"launches": n, "avg_us": t / n * 1e3, "algorithmic_bytes": kind_bytes[k],
                "gbs": kind_bytes[k] / (t / n * 1e-3) / 1e9, "frac_of_hbm_peak": kind_bytes[k] / (t / n * 1e-3) / 1e9 / hbm_peak}
            for k, (n, t) in per_kind.items() if n}
        # in-chain spans of the same stages (a product's span is its GEMM launch; gate_up adds the SwiGLU consumer)
        d = chain["draft"]
        span = lambda *names: sum(d[n][1] for n in names if n in d) / max(max((d[n][0] for n in names if n in d), default=1), 1)
        chain_kind = {"fc": ("gemm_fc",), "qkv": ("gemm_qkv",), "attention": ("attn_tc", "attn_mma", "attn_combine_bf16"),
                      "o": ("gemm_o",), "gate_up": ("gemm_gate_up", "splitk_swiglu"), "down": ("gemm_down",),
                      "lm_head": ("gemm_lm_head",)}
        for k, names in chain_kind.items():
            if k in line["kernels"] and any(n in d for n in names):
                us = span(*names)
                line["kernels"][k]["in_chain_us"] = us
                line["kernels"][k]["in_chain_frac_of_hbm_peak"] = kind_bytes[k] / (us * 1e-6) / 1e9 / hbm_peak
        line["chain_us_per_launch"] = {ph: {n: round(c[1] / c[0], 2) for n, c in sorted(v.items())} for ph, v in chain.items()}
        if with_target and chain["target"]:
            t = chain["target"]
            per_layer = ("gemm_qkv", "rope_append", "attn_tc", "attn_mma", "attn_combine_bf16", "gemm_o", "reduce_norm",
                         "gemm_gate_up", "splitk_swiglu", "gemm_down")
            line["target_layer_in_chain_us"] = sum(t[n][1] for n in per_layer if n in t) / (n_chain * n_layers)
        line["kernels_note"] = ("avg_us: each stage of the draft steps between two CUDA events of its own (isolated: no overlap "
                                "with its neighbours); in_chain_us: the same stage inside the chain of dependent launches, from "
                                "device timestamps taken when each launch's wait for its predecessor returns (span to the next "
                                "launch's); gate_up includes the SwiGLU, attention its combine kernel; bytes = weights (or K/V) only")
        if not args.no_cpu_baseline and world == 1:
            from oracle import poss_oracle as po
            wr = ps.make_weights(cfg, seed)
            kvw = po.widen(ps.make_draft_kv(cfg, seed, cap), np.float32)
            num = po.Num(np.float32, "bf16")
            t0 = time.perf_counter()
            po.draft_round(cfg, wr, kvw, cfg.prefix, tok_h, feat_h, cfg.depth, cfg.topk, cfg.total, num)
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": dt * 1e6, "unit": "us", "cores": len(os.sched_getaffinity(0)),
                                    "kind": "oracle", "sample": "one full draft round of the same workload"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
