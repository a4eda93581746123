#!/usr/bin/env python
"""Benchmark of the tree-verification step (tree attention + acceptance) on B200.

One *step* = ``eagle_tree_verify_attn`` (planner, split-KV attention, combine) followed by
``eagle_tree_accept`` for one batch of synthetic input, on one stream.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

* ``value``: whole-job verify-steps/s with the inputs resident in HBM (device-timed with CUDA events, max
  over ranks).  With N > 1 every rank runs its own batch (no data-path collective: the path shards by
  sequence), so per-GPU work is fixed ("weak").
* ``e2e``: the same step driven from pinned HOST buffers: every step copies its inputs host->device, runs
  the two C-ABI calls and reads the results back.
* ``roofline``: the split-KV attention kernel alone, timed live with CUDA events around that kernel inside
  the timed region, against the measured HBM copy bandwidth.
* ``cpu_baseline``: the fp64 oracle, as it stands, on a bounded sample of the same workload.
* ``--impl reference``: the oracle arm (CPU); rank 0 only.
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
from pathlib import Path

import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2401_15077_b200 import workloads as W  # noqa: E402

METRIC = "tree_verify_steps_per_s"
UNIT = "steps/s"
HBM_FALLBACK_GBS = 6650.0
L2_BYTES = 126 * 2 ** 20
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, from the ncu captures summarised in
# profiles/attn_kernel_serving_mix_b16.md, keyed by (workload, batch); None where no capture exists.
# Full serving_mix: 1180.8 MB read + 24.7 MB written, captured at full size with a one-pass metric list;
# batch 16: 313.0 MB + 8.9 MB from the --set full capture.
NCU_TRAFFIC_BYTES = {("serving_mix", 64): 1_180_839_168 + 24_708_608, ("serving_mix", 16): 313_012_224 + 8_916_992}


def measured_hbm_peak():
    f = ROOT / "MEASURED_PEAKS.json"
    try:
        return float(json.loads(f.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback (profiling recipe, 6.65 TB/s)"


def measured_tensor_peak(long_run: bool):
    """bf16 tensor peak: the sustained figure for a kernel timed inside a long run, the burst figure otherwise."""
    f = ROOT / "MEASURED_PEAKS.json"
    key = "bf16_tflops_sustained" if long_run else "bf16_tflops"
    try:
        return float(json.loads(f.read_text())[key]), f"measured (MEASURED_PEAKS.json {key})"
    except Exception:
        return (1400.0, "fallback (profiling recipe, 1.4 PFLOP/s sustained)") if long_run else \
               (1590.0, "fallback (profiling recipe, 1.59 PFLOP/s)")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def mark(self):
        """Number of samples taken so far (to cut out the samples of the timed region)."""
        return len(self.rows)

    def stop(self, first=0, last=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        window = self.rows[first:last] or self.rows[-3:]
        for r in window:
            try:
                sm.append(float(r[0]))
                smax = float(r[1])
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def host_inputs(cfg, salt, rho):
    attn = W.make_attn_inputs(cfg, salt=salt)
    acc = W.make_accept_inputs(cfg, salt=salt, rho=rho, trees=(attn.tree_sizes, attn.tree_parent))
    return attn, acc


def oracle_step_sample(attn, acc, budget_s, max_seqs=None):
    """Runs the oracle sequence by sequence (attention + acceptance) until ``budget_s`` is spent.
    Returns (sequences done, seconds)."""
    import oracle
    oracle.build()
    B = attn.cfg.batch
    done, t0 = 0, time.perf_counter()
    for b in range(B if max_seqs is None else min(B, max_seqs)):
        s = slice(b, b + 1)
        end = int(attn.seq_lens[b] + attn.tree_sizes[b])
        oracle.tree_verify_attn(attn.q[s], attn.k_cache[s, :, :end].contiguous(), attn.v_cache[s, :, :end].contiguous(),
                                attn.seq_lens[s], attn.tree_parent[s], attn.tree_sizes[s])
        oracle.tree_accept(acc.target_probs[s], acc.draft_probs[s], acc.draft_tokens[s], acc.tree_parent[s],
                           acc.uniforms[s], tree_sizes=acc.tree_sizes[s], greedy=acc.greedy[s])
        done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    return done, time.perf_counter() - t0, oracle.num_threads()


def run_reference(args, cfg, rank, world):
    if rank != 0:
        return
    attn, acc = host_inputs(cfg, 0, args.rho)
    per_step = max(1, min(cfg.batch, args.ref_seqs))
    for _ in range(args.warmup if args.warmup < 2 else 1):
        oracle_step_sample(attn, acc, 1e9, per_step)
    t0 = time.perf_counter()
    cores = 1
    for _ in range(args.steps):
        _, _, cores = oracle_step_sample(attn, acc, 1e9, per_step)
    dt = time.perf_counter() - t0
    value = args.steps * (per_step / cfg.batch) / dt
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "batch": cfg.batch, "rho": args.rho},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"each step runs the first {per_step} of {cfg.batch} sequences (attention + acceptance); "
                                       "value scaled to whole batches"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="serving_mix", choices=list(W.CONFIGS))
    ap.add_argument("--rho", type=float, default=0.9, help="target/draft logit correlation of the synthetic acceptance inputs")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--ref-seqs", type=int, default=1, help="sequences per step of the reference arm")
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling captures on a smaller case)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    cfg = W.CONFIGS[args.workload]
    if args.batch > 0:
        cfg = W.scaled(cfg, batch=args.batch)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return

    import torch.distributed as dist
    from paper_2401_15077_b200 import binding as E, build, replicas
    if rank == 0 or world == 1:
        build.build()
    E.load()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    attn, acc = host_inputs(cfg, replicas.rank_salt(rank), args.rho)
    alg_bytes, alg_flops = attn.algorithmic_bytes(), attn.algorithmic_flops()

    # ---- device-resident input sets; rotate over R sets so that consecutive steps never hit a warm L2
    step_bytes = sum(t.numel() * t.element_size() for t in (attn.k_cache, attn.v_cache))
    touched = alg_bytes
    R = 1 if touched > 2 * L2_BYTES else int(min(48, -(-(1 << 30) // max(touched, 1))))
    host = dict(q=attn.q, k=attn.k_cache, v=attn.v_cache, sl=attn.seq_lens, par=attn.tree_parent, ts=attn.tree_sizes,
                tp=acc.target_probs, dp=acc.draft_probs, tok=acc.draft_tokens, un=acc.uniforms, gr=acc.greedy)
    sets = [{k: v.to(dev) for k, v in host.items()} for _ in range(R)]
    B, T = cfg.batch, cfg.max_tree
    out = torch.empty_like(sets[0]["q"])
    ws = E.alloc_workspace(sets[0]["q"], sets[0]["k"], args.num_splits)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    path = torch.empty((B, T), dtype=torch.int32, device=dev)
    bonus = torch.empty((B,), dtype=torch.int32, device=dev)
    alen = torch.empty((B,), dtype=torch.int32, device=dev)

    def step(s, events=None):
        E.eagle_tree_verify_attn(s["q"], s["k"], s["v"], s["sl"], s["par"], out, tree_sizes=s["ts"], workspace=ws,
                                 status=status, num_splits=args.num_splits, events=events)
        E.eagle_tree_accept(s["tp"], s["dp"], s["tok"], s["par"], s["un"], path, bonus, tree_sizes=s["ts"], greedy=s["gr"],
                            accept_len=alen, status=status)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # started early: nvidia-smi needs a while before its first sample
    for i in range(max(args.warmup, 3)):
        step(sets[i % R])
    torch.cuda.synchronize()
    assert int(status.item()) == 0, E.status_string(int(status.item()))

    K = args.steps
    ev_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in ev_pairs:   # create the underlying CUDA events before handing their handles to the library
        a.record()
        b.record()
    ev_acc = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = E.launch_count()
    barrier()
    if rank == 0 and sampler.mark() == 0:
        time.sleep(0.5)
    m0 = sampler.mark()
    start.record()
    for i in range(K):
        step(sets[(args.warmup + i) % R], ev_pairs[i])
    stop.record()
    barrier()
    clocks = sampler.stop(m0, sampler.mark() + 1) if rank == 0 else None
    launches = E.launch_count() - launches0
    elapsed_ms = start.elapsed_time(stop)
    attn_ms = statistics.mean(a.elapsed_time(b) for a, b in ev_pairs)
    assert int(status.item()) == 0
    elapsed_ms = replicas.max_over_ranks(elapsed_ms, dev)
    value = world * K / (elapsed_ms * 1e-3)

    # ---- acceptance alone (reported, not part of the headline)
    for i in range(min(K, 10)):
        s = sets[i % R]
        ev_acc[i][0].record()
        E.eagle_tree_accept(s["tp"], s["dp"], s["tok"], s["par"], s["un"], path, bonus, tree_sizes=s["ts"], greedy=s["gr"],
                            accept_len=alen, status=status)
        ev_acc[i][1].record()
    torch.cuda.synchronize()
    accept_ms = statistics.mean(ev_acc[i][0].elapsed_time(ev_acc[i][1]) for i in range(min(K, 10)))
    mean_tokens = float(alen.float().mean().item()) + 1.0

    # ---- the same acceptance on logits (softmax fused into the walk; reported, not part of the headline).  The logits are
    # the logarithms of the step's probabilities, so at temperature 1 the walk must return the same tokens.
    s = sets[0]
    path_p, bonus_p = path.clone(), bonus.clone()
    zt, zd = s["tp"].clamp_min(1e-37).log(), s["dp"].clamp_min(1e-37).log()
    path_l, bonus_l = torch.empty_like(path), torch.empty_like(bonus)
    l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    E.eagle_tree_accept_logits(zt, zd, s["tok"], s["par"], s["un"], 1.0, path_l, bonus_l, tree_sizes=s["ts"], greedy=s["gr"], status=status)
    l0.record()
    for i in range(5):
        E.eagle_tree_accept_logits(zt, zd, s["tok"], s["par"], s["un"], 1.0, path_l, bonus_l, tree_sizes=s["ts"], greedy=s["gr"],
                                   status=status)
    l1.record()
    torch.cuda.synchronize()
    accept_logits_ms = l0.elapsed_time(l1) / 5
    logits_same = int(((path_l == path_p).all(dim=1) & (bonus_l == bonus_p)).sum().item())
    del zt, zd

    # ---- child selection for the next drafting pass (App. A.1; reported, not part of the headline): 4 children for each
    # of the first 8 nodes' draft rows of every sequence (top-4 for greedy sequences, 4 draws otherwise)
    s = sets[0]
    R_exp, K_exp = min(8, T), 4
    rows_exp = s["dp"][:, :R_exp].contiguous()
    nc_exp = torch.full((B, R_exp), K_exp, dtype=torch.int32, device=dev)
    un_exp = torch.rand((B, R_exp, K_exp), device=dev)
    x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    E.eagle_tree_expand(rows_exp, nc_exp, K_exp, uniforms=un_exp, greedy=s["gr"], status=status)
    x0.record()
    for i in range(10):
        E.eagle_tree_expand(rows_exp, nc_exp, K_exp, uniforms=un_exp, greedy=s["gr"], status=status)
    x1.record()
    torch.cuda.synchronize()
    expand_ms = x0.elapsed_time(x1) / 10
    expand_bytes = rows_exp.numel() * 4
    del rows_exp

    # ---- the same attention over a paged cache (reported, not part of the headline): the first input set's keys and
    # values cut into pages of 128 and of 16 slots, scattered over the pool by a seeded permutation
    s = sets[0]
    step(s)
    ref_bits = out.view(torch.int16).clone()
    paged = {}
    for ps in (128, 16):
        cap_p = (s["k"].shape[2] + ps - 1) // ps * ps
        per_seq = cap_p // ps

        def to_pages(x):
            xp = torch.nn.functional.pad(x, (0, 0, 0, cap_p - x.shape[2]))
            return xp.view(B, cfg.num_kv_heads, per_seq, ps, cfg.head_dim).permute(0, 2, 1, 3, 4).reshape(B * per_seq, cfg.num_kv_heads,
                                                                                                      ps, cfg.head_dim)
        gperm = torch.Generator().manual_seed(W.seed_for(cfg.index, "pages", ps))
        perm = torch.randperm(B * per_seq, generator=gperm).to(dev)       # page i of the ordered pool goes to pool slot perm[i]
        shape = (B * per_seq, cfg.num_kv_heads, ps, cfg.head_dim)
        kp, vp = torch.empty(shape, dtype=torch.bfloat16, device=dev), torch.empty(shape, dtype=torch.bfloat16, device=dev)
        kp[perm], vp[perm] = to_pages(s["k"]), to_pages(s["v"])
        table = perm.view(B, per_seq).to(torch.int32).contiguous()
        pe = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(8)]
        for e in pe:
            for x in e:
                x.record()
        for e in pe:
            E.eagle_tree_verify_attn_paged(s["q"], kp, vp, table, s["sl"], s["par"], out, tree_sizes=s["ts"], workspace=ws,
                                           status=status, num_splits=args.num_splits, events=(e[0], e[1]))
        torch.cuda.synchronize()
        paged[f"page_{ps}"] = {"attn_kernel_ms": statistics.median(e[0].elapsed_time(e[1]) for e in pe[3:]),
                               "same_bits_as_contiguous": bool(torch.equal(out.view(torch.int16), ref_bits))}
        del kp, vp
    del ref_bits
    assert int(status.item()) == 0

    # ---- commit of the accepted path for this layer's cache (the step after verification; reported, not part of the
    # headline).  It moves rows in place, so it runs on the last input set, after everything that reads the cache.
    s = sets[-1]
    new_len = torch.empty((B,), dtype=torch.int32, device=dev)
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        E.eagle_tree_commit(s["k"], s["v"], s["sl"], path, T, new_seq_lens=new_len, status=status)
    torch.cuda.synchronize()
    c0.record()
    for i in range(50):
        E.eagle_tree_commit(s["k"], s["v"], s["sl"], path, T, new_seq_lens=new_len, status=status)
    c1.record()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    commit_ms = c0.elapsed_time(c1) / 50      # back-to-back calls: the larger of kernel time and enqueue time per call
    moved = int(((path >= 0) & (path != torch.arange(T, device=dev, dtype=torch.int32)[None, :])).sum().item())
    commit_bytes = moved * cfg.num_kv_heads * cfg.head_dim * 2 * 2 * 2     # rows that change slot: K and V, read + written

    # ---- end to end from pinned host buffers, through the library's host-buffer entry point: every step copies all
    # inputs host->device, runs attention + acceptance, and copies the results back
    pinned = dict(q=attn.q, k_cache=attn.k_cache, v_cache=attn.v_cache, seq_lens=attn.seq_lens, tree_sizes=attn.tree_sizes,
                  tree_parent=attn.tree_parent, target_probs=acc.target_probs, draft_probs=acc.draft_probs,
                  draft_tokens=acc.draft_tokens, uniforms=acc.uniforms, greedy=acc.greedy)
    pinned = {k: v.pin_memory() for k, v in pinned.items()}
    del sets
    torch.cuda.empty_cache()
    runner = E.HostStepRunner(pinned, dev)
    h2d, d2h = runner.h2d_bytes, runner.d2h_bytes
    runner.run()
    barrier()
    assert int(runner.status.item()) == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        runner.run()
    e1.record()
    barrier()
    e2e_value = world * args.e2e_steps / (replicas.max_over_ranks(e0.elapsed_time(e1), dev) * 1e-3)
    # the step driven from host buffers gives the same tokens as the device-resident one (all input sets hold the same data)
    same_tokens = bool(torch.equal(runner.bonus_token, bonus.cpu()))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # which roof is lower for this workload: moving the algorithmic bytes at the measured copy bandwidth, or doing the
    # algorithmic flops (4 * visible keys * tree nodes * query heads * head_dim, no padding) at the measured bf16 rate
    hbm_peak, hbm_src = measured_hbm_peak()
    tc_peak, tc_src = measured_tensor_peak(K >= 200)
    hbm_achieved = alg_bytes / (attn_ms * 1e-3) / 1e9
    tc_achieved = alg_flops / (attn_ms * 1e-3) / 1e12
    tensor_bound = alg_flops / (tc_peak * 1e12) > alg_bytes / (hbm_peak * 1e9)
    if tensor_bound:
        bound, achieved, peak, peak_src, roof_unit = "tensor", tc_achieved, tc_peak, tc_src, "TFLOP/s"
    else:
        bound, achieved, peak, peak_src, roof_unit = "hbm", hbm_achieved, hbm_peak, hbm_src, "GB/s"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": B, "num_q_heads": cfg.num_q_heads, "num_kv_heads": cfg.num_kv_heads,
                   "head_dim": cfg.head_dim, "prefix": list(cfg.prefix), "tree": list(cfg.tree), "vocab": cfg.vocab,
                   "greedy": cfg.greedy, "rho": args.rho, "parallelism": f"replicas x{world}",
                   "l2": (f"rotating over {R} input sets" if R > 1 else "inputs larger than L2 (single set)")},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
                "h2d_whole_tensor_bytes": runner.full_h2d_bytes,
                "api": "eagle_tree_verify_step_host", "same_tokens_as_device_path": same_tokens},
        "roofline": {"bound": bound, "kernel": "split-KV tree attention", "achieved": achieved, "peak": peak, "unit": roof_unit,
                     "frac": achieved / peak, "peak_source": peak_src, "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, cfg.batch)),
                     "algorithmic_bytes": alg_bytes, "algorithmic_flops": alg_flops, "ms_per_launch": attn_ms,
                     "gbs": hbm_achieved, "hbm_frac": hbm_achieved / hbm_peak, "tflops": tc_achieved, "tensor_frac": tc_achieved / tc_peak},
        "breakdown": {"attn_kernel_ms": attn_ms, "accept_ms": accept_ms, "tokens_per_step": mean_tokens,
                      "sequence_steps_per_s": value * B,
                      "accept_on_logits": {"ms": accept_logits_ms, "temperature": 1.0,
                                           "sequences_with_the_same_tokens_as_on_probabilities": logits_same, "of": B},
                      "tree_expand": {"ms": expand_ms, "rows": B * R_exp, "children": K_exp, "bytes": expand_bytes,
                                      "gbs": expand_bytes / (expand_ms * 1e-3) / 1e9,
                                      "note": "back-to-back calls on the same rows (warm L2)"},
                      "paged_attention": paged,
                      "kv_commit": {"ms": commit_ms, "rows_moved_per_kv_head": moved, "bytes": commit_bytes,
                                    "gbs": commit_bytes / (commit_ms * 1e-3) / 1e9, "bound": "launch + memory latency"}},
    }
    if not args.no_cpu_baseline:
        done, secs, cores = oracle_step_sample(attn, acc, args.cpu_budget)
        line["cpu_baseline"] = {"value": (done / B) / secs, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {done} of {B} sequences of the same batch (attention + acceptance), "
                                          f"{secs:.1f} s; value scaled to whole batches"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
