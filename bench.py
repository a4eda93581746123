#!/usr/bin/env python
"""Benchmark of the tree-verification step (tree attention + acceptance) on B200.

One *step* = ``eagle_tree_verify_attn`` (planner, split-KV attention, combine) followed by
``eagle_tree_accept`` for one batch of synthetic input, on one stream.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

* ``value``: whole-job verify-steps/s with the inputs resident in HBM (device-timed with CUDA events, max
  over ranks).  With N > 1 every rank runs its own batch (no data-path collective: the path shards by
  sequence), so per-GPU work is fixed ("weak").  Started without a launcher and with ``--gpus N`` > 1 the
  script starts its N ranks itself (torch.distributed.run on 127.0.0.1).
* ``e2e``: the same step driven from pinned HOST buffers: every step copies its inputs host->device, runs
  the two C-ABI calls and reads the results back.
* ``roofline``: the split-KV attention kernel alone, timed live with CUDA events around that kernel inside
  the timed region, against the measured HBM copy bandwidth (or the measured bf16 rate where that binds).
* ``breakdown.sustained``: the same step back to back for seconds, with the SM clock sampled meanwhile.
* ``breakdown.workloads``: the other configurations (70B-, Mixtral-, 7B-shaped, tiny), a few dozen steps each.
* ``breakdown.per_layer``: one plan for the verification pass, then attention + combine per layer (also as one CUDA graph).
* ``cpu_baseline`` / ``parity``: the fp64 oracle, as it stands, on a bounded sample of the same workload; its
  outputs are compared with the device path's on the way.
* ``--impl reference``: the oracle arm (CPU); rank 0 only.
"""
from __future__ import annotations

import argparse
import hashlib
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
HBM_NOMINAL_GBS = 8000.0
L2_BYTES = 126 * 2 ** 20
SM_COUNT, EX2_PER_SM_PER_CLK = 148, 16      # special-function rate behind the exponentials' bound
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch from the ncu captures summarised in
# profiles/attn_kernel_serving_mix_b16.md, keyed by (workload, batch), with the SHA-256 of the attention kernel's source
# the captures were taken on: when the source has changed since, the figure is stale and `traffic` is reported as null.
NCU_TRAFFIC = {
    "attn_cu_sha256": "45abb4aec25ea42f4cba9b9c12940521db7b31208c3f05b689e433d667c06e1e",
    # full size: one-pass metric list, two launches averaged (1176.3 MB read + 22.8 MB written); batch 16: --set full
    # (taken before the epilogue's stores changed; the reads it measures did not)
    "bytes": {("serving_mix", 64): 1_176_343_168 + 22_765_312, ("serving_mix", 16): 313_046_528 + 9_554_304},
}


def ncu_traffic(cfg):
    src = ROOT / "paper_2401_15077_b200" / "csrc" / "attn.cu"
    try:
        current = hashlib.sha256(src.read_bytes()).hexdigest()
    except OSError:
        current = None
    value = NCU_TRAFFIC["bytes"].get((cfg.name, cfg.batch))
    if value is None:
        return None, "no capture for this workload"
    if current != NCU_TRAFFIC["attn_cu_sha256"]:
        return None, "stale: the attention kernel's source changed after the ncu capture"
    return value, "ncu capture on this source (profiles/attn_kernel_serving_mix_b16.md)"


def peaks():
    f = ROOT / "MEASURED_PEAKS.json"
    try:
        d = json.loads(f.read_text())
        return {"hbm": float(d["hbm_gbs"]), "tc_burst": float(d["bf16_tflops"]), "tc_sustained": float(d["bf16_tflops_sustained"]),
                "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured (MEASURED_PEAKS.json)"}
    except Exception:
        return {"hbm": HBM_FALLBACK_GBS, "tc_burst": 1590.0, "tc_sustained": 1400.0, "sm_max_mhz": 1965.0,
                "source": "fallback (profiling recipe: 6.65 TB/s, 1.59 / 1.4 PFLOP/s)"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi (a read-only query) while the timed region runs."""
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
        """Number of samples taken so far (to cut out the samples of a timed region)."""
        return len(self.rows)

    def window(self, first=0, last=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        sm, smax, power, reasons = [], None, [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in (self.rows[first:last] or self.rows[-3:]):
            try:
                sm.append(float(r[0]))
                smax = float(r[1])
                power.append(float(r[2]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm), "power_w": statistics.median(power) if power else None}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()


def host_inputs(cfg, salt, rho):
    attn = W.make_attn_inputs(cfg, salt=salt)
    acc = W.make_accept_inputs(cfg, salt=salt, rho=rho, trees=(attn.tree_sizes, attn.tree_parent))
    return attn, acc


def seq_work(attn):
    """Relative cost of each sequence for the oracle: visible keys x tree nodes (its attention dominates)."""
    return ((attn.seq_lens.long() + attn.tree_sizes.long()) * attn.tree_sizes.long()).double()


def oracle_step_sample(attn, acc, budget_s, max_seqs=None, keep=False):
    """Runs the oracle sequence by sequence (attention + acceptance) until ``budget_s`` is spent.
    Returns (sequences done, seconds, threads, outputs of the sequences done when ``keep``)."""
    import oracle
    oracle.build()
    B = attn.cfg.batch
    done, kept, t0 = 0, [], time.perf_counter()
    for b in range(B if max_seqs is None else min(B, max_seqs)):
        s = slice(b, b + 1)
        end = int(attn.seq_lens[b] + attn.tree_sizes[b])
        o = oracle.tree_verify_attn(attn.q[s], attn.k_cache[s, :, :end].contiguous(), attn.v_cache[s, :, :end].contiguous(),
                                    attn.seq_lens[s], attn.tree_parent[s], attn.tree_sizes[s])
        r = oracle.tree_accept(acc.target_probs[s], acc.draft_probs[s], acc.draft_tokens[s], acc.tree_parent[s],
                               acc.uniforms[s], tree_sizes=acc.tree_sizes[s], greedy=acc.greedy[s])
        if keep:
            kept.append((o, r))
        done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    return done, time.perf_counter() - t0, oracle.num_threads(), kept


def scaled_steps_per_s(attn, done, secs):
    """Whole-batch steps/s from a sample of the first ``done`` sequences, scaled by their share of the batch's work."""
    w = seq_work(attn)
    share = float(w[:done].sum() / w.sum()) if float(w.sum()) > 0 else done / attn.cfg.batch
    return share / secs, share


def run_reference(args, cfg, rank, world):
    """The oracle arm: every step is the whole batch (attention + acceptance of every sequence) unless --ref-seqs limits it."""
    if rank != 0:
        return
    attn, acc = host_inputs(cfg, 0, args.rho)
    per_step = cfg.batch if args.ref_seqs <= 0 else max(1, min(cfg.batch, args.ref_seqs))
    for _ in range(1 if args.warmup > 0 else 0):       # one warm-up pass is enough for a CPU program (pages in the inputs)
        oracle_step_sample(attn, acc, 1e9, per_step)
    t0 = time.perf_counter()
    cores = 1
    for _ in range(args.steps):
        _, _, cores, _ = oracle_step_sample(attn, acc, 1e9, per_step)
    dt = time.perf_counter() - t0
    value, share = scaled_steps_per_s(attn, per_step, dt / args.steps)
    sample = (f"every step runs all {cfg.batch} sequences (attention + acceptance)" if per_step == cfg.batch else
              f"each step runs the first {per_step} of {cfg.batch} sequences ({share:.3f} of the batch's work); value scaled to whole batches")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "impl": "reference", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": 1 if args.warmup > 0 else 0, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "batch": cfg.batch, "rho": args.rho},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


class StepContext:
    """Device-resident inputs of one workload (rotated over R sets so that no step finds its inputs in L2) and the step."""

    def __init__(self, E, cfg, dev, salt, rho, num_splits):
        self.E, self.cfg, self.dev, self.num_splits = E, cfg, dev, num_splits
        self.attn, self.acc = host_inputs(cfg, salt, rho)
        attn, acc = self.attn, self.acc
        self.alg_bytes, self.alg_flops = attn.algorithmic_bytes(), attn.algorithmic_flops()
        self.alg_exps = self.alg_flops // (4 * cfg.head_dim)
        self.R = 1 if self.alg_bytes > 2 * L2_BYTES else int(min(48, -(-(1 << 30) // max(self.alg_bytes, 1))))
        host = dict(q=attn.q, k=attn.k_cache, v=attn.v_cache, sl=attn.seq_lens, par=attn.tree_parent, ts=attn.tree_sizes,
                    tp=acc.target_probs, dp=acc.draft_probs, tok=acc.draft_tokens, un=acc.uniforms, gr=acc.greedy)
        self.sets = [{k: v.to(dev) for k, v in host.items()} for _ in range(self.R)]
        B, T = cfg.batch, cfg.max_tree
        s0 = self.sets[0]
        self.out = torch.empty_like(s0["q"])
        self.ws = E.alloc_workspace(s0["q"], s0["k"], num_splits)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.path = torch.empty((B, T), dtype=torch.int32, device=dev)
        self.bonus = torch.empty((B,), dtype=torch.int32, device=dev)
        self.alen = torch.empty((B,), dtype=torch.int32, device=dev)

    def accept(self, s):
        self.E.eagle_tree_accept(s["tp"], s["dp"], s["tok"], s["par"], s["un"], self.path, self.bonus, tree_sizes=s["ts"],
                                 greedy=s["gr"], accept_len=self.alen, status=self.status)

    def step(self, i, events=None):
        s = self.sets[i % self.R]
        self.E.eagle_tree_verify_attn(s["q"], s["k"], s["v"], s["sl"], s["par"], self.out, tree_sizes=s["ts"], workspace=self.ws,
                                      status=self.status, num_splits=self.num_splits, events=events)
        self.accept(s)

    def check(self):
        code = int(self.status.item())
        assert code == 0, self.E.status_string(code)

    def timed(self, K, first=0, every=1):
        """K steps back to back; the attention kernel of every ``every``-th step is timed by the library's own events.
        Returns (elapsed ms, mean attention-kernel ms, launches)."""
        n_ev = (K + every - 1) // every
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
        for a, b in evs:        # create the underlying CUDA events before handing their handles to the library
            a.record()
            b.record()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = self.E.launch_count()
        torch.cuda.synchronize()
        start.record()
        for i in range(K):
            self.step(first + i, evs[i // every] if i % every == 0 else None)
        stop.record()
        torch.cuda.synchronize()
        return start.elapsed_time(stop), statistics.mean(a.elapsed_time(b) for a, b in evs), self.E.launch_count() - launches0

    def graph_leg(self, K=50):
        """The same step captured once in a CUDA graph (all R input sets in turn, so that no replay finds its inputs in L2) and
        replayed: what the step costs without the host's launch gaps."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            for i in range(self.R):
                self.step(i)                       # (every first-call set-up of the library has long happened)
            side.synchronize()
            with torch.cuda.graph(g, stream=side):
                for i in range(self.R):
                    self.step(i)
        torch.cuda.current_stream().wait_stream(side)
        reps = max(1, K // self.R)
        for _ in range(2):
            g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        self.check()
        ms = a.elapsed_time(b) / (reps * self.R)
        return {"ms_per_step": ms, "steps_per_s": 1e3 / ms, "steps": reps * self.R,
                "note": "the four launches of a step replayed from one CUDA graph"}

    def per_layer(self, layers=32):
        """One plan for the verification pass, then attention + combine for each of ``layers`` layers (rotating K/V sets)."""
        s0 = self.sets[0]
        cfg = self.cfg
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]

        def one_pass():
            plan = self.E.eagle_tree_verify_plan(tuple(s0["q"].shape), cfg.num_kv_heads, s0["k"].shape[2], s0["sl"], s0["par"],
                                                 tree_sizes=s0["ts"], num_splits=self.num_splits, workspace=self.ws, status=self.status)
            e[1].record()
            for l in range(layers):
                s = self.sets[l % self.R]
                plan.attend(s["q"], s["k"], s["v"], self.out, status=self.status)

        one_pass()
        torch.cuda.synchronize()
        e[0].record()
        one_pass()
        e[2].record()
        torch.cuda.synchronize()
        out = {"layers": layers, "plan_ms": e[0].elapsed_time(e[1]), "ms_per_layer": e[1].elapsed_time(e[2]) / layers,
               "note": "eagle_tree_verify_plan once, then eagle_tree_verify_attn_planned per layer"}
        # the same pass (plan + every layer's attention and combine) captured in one CUDA graph and replayed: the host's
        # launch gaps are gone, which is what a serving loop that replays its forward pass sees
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            side.synchronize()
            with torch.cuda.graph(g, stream=side):
                one_pass_plain = self.E.eagle_tree_verify_plan(tuple(s0["q"].shape), cfg.num_kv_heads, s0["k"].shape[2], s0["sl"], s0["par"],
                                                               tree_sizes=s0["ts"], num_splits=self.num_splits, workspace=self.ws,
                                                               status=self.status)
                for l in range(layers):
                    s = self.sets[l % self.R]
                    one_pass_plain.attend(s["q"], s["k"], s["v"], self.out, status=self.status)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        g.replay()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        self.check()
        out["graph_ms_per_layer"] = a.elapsed_time(b) / (2 * layers)
        out["graph_note"] = "plan + %d layers replayed from one CUDA graph; the plan's share is included" % layers
        return out

    def fp8_leg(self, attn_ms_bf16, pk, calls=12):
        """The same attention over the same cache stored as fp8 (e4m3) codes with a scale per (sequence, KV head): the
        attention kernel's time (library events), against the bf16 call's, and its own HBM fraction (half the cache bytes)."""
        cfg = self.cfg
        if cfg.head_dim != 128:
            return None
        f8 = W.make_fp8_cache(self.attn)
        dev, s = self.dev, self.sets[0]
        sets = [(f8.k_codes.to(dev), f8.v_codes.to(dev)) for _ in range(max(1, min(self.R, 24)))]
        ks, vs = f8.k_scale.to(dev), f8.v_scale.to(dev)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(calls)]
        for a, b in evs:
            a.record()
            b.record()
        for i in range(3 + calls):
            kc, vc = sets[i % len(sets)]
            self.E.eagle_tree_verify_attn_fp8(s["q"], kc, vc, ks, vs, s["sl"], s["par"], self.out, tree_sizes=s["ts"], workspace=self.ws,
                                              status=self.status, num_splits=self.num_splits, events=evs[i - 3] if i >= 3 else None)
        torch.cuda.synchronize()
        self.check()
        ms = statistics.mean(a.elapsed_time(b) for a, b in evs)
        kv_rows = int((self.attn.seq_lens.long() + self.attn.tree_sizes.long()).sum()) * cfg.num_kv_heads
        alg = kv_rows * cfg.head_dim * 2 + int(self.attn.tree_sizes.long().sum()) * cfg.num_q_heads * cfg.head_dim * 4 + \
            2 * 4 * cfg.batch * cfg.num_kv_heads
        gbs = alg / (ms * 1e-3) / 1e9
        res = {"attn_kernel_ms": ms, "ratio_to_bf16": ms / attn_ms_bf16, "algorithmic_bytes": alg, "gbs": gbs, "hbm_frac": gbs / pk["hbm"],
               "note": "e4m3 codes + fp32 scale per (sequence, KV head); codes widened exactly to fp16 in shared memory, fp16 x fp16 MMAs"}
        # the same codes kept in pages of 64 slots scattered over a pool (one set: this is a reported side figure)
        flat_bits = self.out.view(torch.int16).clone()      # the last timed call read sets[(2 + calls) % len(sets)]: all sets are equal
        kc, vc = sets[0]
        B, ps = cfg.batch, 64
        cap_p = (kc.shape[2] + ps - 1) // ps * ps
        per_seq = cap_p // ps

        def to_pages(x):
            xp = torch.nn.functional.pad(x, (0, 0, 0, cap_p - x.shape[2]), value=0x7F)
            return xp.view(B, cfg.num_kv_heads, per_seq, ps, cfg.head_dim).permute(0, 2, 1, 3, 4).reshape(
                B * per_seq, cfg.num_kv_heads, ps, cfg.head_dim)
        perm = torch.randperm(B * per_seq, generator=torch.Generator().manual_seed(W.seed_for(cfg.index, "pages", ps))).to(dev)
        shape = (B * per_seq, cfg.num_kv_heads, ps, cfg.head_dim)
        kp, vp = torch.empty(shape, dtype=torch.uint8, device=dev), torch.empty(shape, dtype=torch.uint8, device=dev)
        kp[perm], vp[perm] = to_pages(kc), to_pages(vc)
        table = perm.view(B, per_seq).to(torch.int32).contiguous()
        pe = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(8)]
        for a, b in pe:
            a.record()
            b.record()
        for e in pe:
            self.E.eagle_tree_verify_attn_paged_fp8(s["q"], kp, vp, ks, vs, table, s["sl"], s["par"], self.out, tree_sizes=s["ts"],
                                                    workspace=self.ws, status=self.status, num_splits=self.num_splits, events=e)
        torch.cuda.synchronize()
        self.check()
        res["paged_64"] = {"attn_kernel_ms": statistics.median(a.elapsed_time(b) for a, b in pe[3:]),
                           "same_bits_as_contiguous_fp8": bool(torch.equal(self.out.view(torch.int16), flat_bits))}
        del kp, vp
        return res

    def free(self):
        self.sets = None
        self.out = self.ws = None
        torch.cuda.empty_cache()


def bounds(ctx, attn_ms, pk, long_run):
    """Times the attention launch cannot beat, and how close it came to the largest of them."""
    tc = pk["tc_sustained"] if long_run else pk["tc_burst"]
    t_hbm = ctx.alg_bytes / (pk["hbm"] * 1e9) * 1e3
    t_mma = ctx.alg_flops / (tc * 1e12) * 1e3
    t_exp = ctx.alg_exps / (SM_COUNT * EX2_PER_SM_PER_CLK * pk["sm_max_mhz"] * 1e6) * 1e3
    name, t = max((("hbm", t_hbm), ("tensor", t_mma), ("alu", t_exp)), key=lambda x: x[1])
    gbs, tfl = ctx.alg_bytes / (attn_ms * 1e-3) / 1e9, ctx.alg_flops / (attn_ms * 1e-3) / 1e12
    return {"attn_kernel_ms": attn_ms, "gbs": gbs, "hbm_frac": gbs / pk["hbm"], "hbm_frac_nominal": gbs / HBM_NOMINAL_GBS,
            "tflops": tfl, "tensor_frac": tfl / tc, "tensor_peak": tc, "t_hbm_ms": t_hbm, "t_mma_ms": t_mma,
            "t_exp_ms": t_exp, "bound": name, "frac_of_binding_bound": t / attn_ms,
            "algorithmic_bytes": ctx.alg_bytes, "algorithmic_flops": ctx.alg_flops}


def parity_record(ctx, gpu_out, gpu_path, gpu_bonus, gpu_alen, kept):
    """The oracle's outputs for the sequences it was timed on, against the device path's for the same inputs."""
    import numpy as np
    from oracle.compare import first_differing_decision
    max_abs, sum_abs, count, mism, tol = 0.0, 0.0, 0, 0, 0
    greedy = ctx.acc.greedy.numpy()
    for b, (o, r) in enumerate(kept):
        n = int(ctx.attn.tree_sizes[b])
        err = np.abs(gpu_out[b, :n].double().numpy() - o[0, :n])
        if err.size:
            max_abs, sum_abs, count = max(max_abs, float(err.max())), sum_abs + float(err.sum()), count + err.size
        same = (np.array_equal(gpu_path[b], r["accepted_path"][0]) and int(gpu_bonus[b]) == int(r["bonus_token"][0]) and
                int(gpu_alen[b]) == int(r["accept_len"][0]))
        if not same:
            d = first_differing_decision(r, 0, gpu_path[b], gpu_bonus[b])
            near = d is not None and float(r["dec_margin"][0, d]) < 1e-5 and not greedy[b]
            tol += 1 if near else 0
            mism += 0 if near else 1
    return {"sequences_checked": len(kept), "attn_max_abs": max_abs, "attn_mean_abs": sum_abs / max(count, 1),
            "attn_bounds": [2e-2, 2e-3], "accept_mismatches": mism, "accept_tolerated": tol,
            "rule": "identical tokens, except a margin below 1e-5 at the first differing decision (counted as tolerated)"}


def self_launch(args):
    """Started bare with --gpus N > 1: start the N ranks (one per GPU) and let rank 0 print the line."""
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), str(Path(__file__).resolve())] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


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
    ap.add_argument("--ref-seqs", type=int, default=0, help="sequences per step of the reference arm (0: the whole batch)")
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustain-seconds", type=float, default=2.5, help="length of the sustained leg (0: skip)")
    ap.add_argument("--other-steps", type=int, default=50, help="timed steps for each of the other workloads (0: skip)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling captures on a smaller case)")
    ap.add_argument("--only-step", action="store_true", help="headline loop only (for profiling captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    cfg = W.CONFIGS[args.workload]
    if args.batch > 0:
        cfg = W.scaled(cfg, batch=args.batch)
    if args.gpus > 1 and "RANK" not in os.environ:
        self_launch(args)
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

    pk = peaks()
    ctx = StepContext(E, cfg, dev, replicas.rank_salt(rank), args.rho, args.num_splits)
    attn, acc, B, T = ctx.attn, ctx.acc, cfg.batch, cfg.max_tree

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()          # started early: nvidia-smi needs a while before its first sample
    warm = max(args.warmup, 3)
    for i in range(warm):
        ctx.step(i)
    torch.cuda.synchronize()
    ctx.check()

    # ---- the headline: K steps, bracketed by a barrier and a device synchronisation on both sides
    K = args.steps
    barrier()
    if rank == 0 and sampler.mark() == 0:
        time.sleep(0.5)
    m0 = sampler.mark()
    elapsed_ms, attn_ms, launches = ctx.timed(K, first=warm)
    barrier()
    clocks = sampler.window(m0, sampler.mark() + 1) if rank == 0 else None
    ctx.check()
    value = replicas.whole_job_steps_per_s(elapsed_ms, K, dev)      # all ranks' steps over the slowest rank's device time
    elapsed_ms = replicas.max_over_ranks(elapsed_ms, dev)
    head = bounds(ctx, attn_ms, pk, K >= 200)

    extras = {}
    if not args.only_step:
        # ---- sustained: the same step back to back for seconds (the power cap settles the clock), clocks sampled meanwhile
        if args.sustain_seconds > 0:
            n_sus = max(K, int(args.sustain_seconds * 1e3 / (elapsed_ms / K)) + 1)
            m1 = sampler.mark()
            sus_ms, sus_attn_ms, _ = ctx.timed(n_sus, first=warm, every=8)
            c = sampler.window(m1, sampler.mark() + 1) if rank == 0 else {"sm_mhz": None}
            sb = bounds(ctx, sus_attn_ms, pk, True)
            extras["sustained"] = {"steps": n_sus, "seconds": sus_ms * 1e-3, "steps_per_s": n_sus / (sus_ms * 1e-3), "ms_per_step": sus_ms / n_sus,
                                   "attn_kernel_us": sus_attn_ms * 1e3, "clocks": c,
                                   "attn_us_x_mhz": (sus_attn_ms * 1e3 * c["sm_mhz"]) if c.get("sm_mhz") else None,
                                   "hbm_frac": sb["hbm_frac"], "hbm_frac_nominal": sb["hbm_frac_nominal"], "tensor_frac": sb["tensor_frac"],
                                   "frac_of_binding_bound": sb["frac_of_binding_bound"], "bound": sb["bound"]}
            ctx.check()

        # ---- acceptance alone (reported, not part of the headline)
        ev_acc = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]
        for i, (a, b) in enumerate(ev_acc):
            a.record()
            ctx.accept(ctx.sets[i % ctx.R])
            b.record()
        torch.cuda.synchronize()
        accept_ms = statistics.mean(a.elapsed_time(b) for a, b in ev_acc)
        path, bonus, alen, status = ctx.path, ctx.bonus, ctx.alen, ctx.status

        # ---- the same acceptance with uncorrelated draft and target logits (rho = 0: rejection-heavy, the longest walks)
        acc0 = W.make_accept_inputs(cfg, salt=replicas.rank_salt(rank), rho=0.0, trees=(attn.tree_sizes, attn.tree_parent))
        t0 = {k: v.to(dev) for k, v in dict(tp=acc0.target_probs, dp=acc0.draft_probs, tok=acc0.draft_tokens, un=acc0.uniforms).items()}
        s0 = ctx.sets[0]
        ev0 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(6)]
        for a, b in ev0:
            a.record()
            E.eagle_tree_accept(t0["tp"], t0["dp"], t0["tok"], s0["par"], t0["un"], path, bonus, tree_sizes=s0["ts"], greedy=s0["gr"],
                                accept_len=alen, status=status)
            b.record()
        torch.cuda.synchronize()
        accept_rho0 = {"ms": statistics.mean(a.elapsed_time(b) for a, b in ev0[1:]), "tokens_per_step": float(alen.float().mean().item()) + 1.0}
        del t0, acc0

        # ---- the device path's outputs on input set 0, kept for the parity record
        ctx.step(0)
        torch.cuda.synchronize()
        gpu_out, gpu_path, gpu_bonus, gpu_alen = ctx.out.cpu(), path.cpu().numpy(), bonus.cpu().numpy(), alen.cpu().numpy()
        mean_tokens = float(alen.float().mean().item()) + 1.0

        # ---- the same acceptance on logits (softmax fused into the walk; reported, not part of the headline).  The logits are
        # the logarithms of the step's probabilities, so at temperature 1 the walk must return the same tokens.
        s = ctx.sets[0]
        path_p, bonus_p = path.clone(), bonus.clone()
        zt, zd = s["tp"].clamp_min(1e-37).log(), s["dp"].clamp_min(1e-37).log()
        path_l, bonus_l = torch.empty_like(path), torch.empty_like(bonus)
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        kw = dict(tree_sizes=s["ts"], greedy=s["gr"], status=status)
        E.eagle_tree_accept_logits(zt, zd, s["tok"], s["par"], s["un"], 1.0, path_l, bonus_l, **kw)
        l0.record()
        for i in range(5):
            E.eagle_tree_accept_logits(zt, zd, s["tok"], s["par"], s["un"], 1.0, path_l, bonus_l, **kw)
        l1.record()
        torch.cuda.synchronize()
        accept_logits_ms = l0.elapsed_time(l1) / 5
        logits_same = int(((path_l == path_p).all(dim=1) & (bonus_l == bonus_p)).sum().item())
        del zt, zd

        # ---- child selection for the next drafting pass (App. A.1; reported, not part of the headline): 4 children for each
        # of the first 8 nodes' draft rows of every sequence (top-4 for greedy sequences, 4 draws otherwise)
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

        # ---- the step replayed from a CUDA graph (no launch gaps)
        cuda_graph = ctx.graph_leg()

        # ---- one plan per verification pass, attention + combine per layer
        per_layer = ctx.per_layer()
        per_layer["attn_kernel_share_of_layer"] = attn_ms / per_layer["ms_per_layer"]

        # ---- the same attention over an fp8 copy of the cache (reported, not part of the headline)
        fp8_kv = ctx.fp8_leg(attn_ms, pk)

        # ---- the same attention over a paged cache (reported, not part of the headline): the first input set's keys and
        # values cut into pages of 128 and of 16 slots, scattered over the pool by a seeded permutation
        ctx.step(0)
        ref_bits = ctx.out.view(torch.int16).clone()
        paged = {}
        for ps in (128, 16):
            cap_p = (s["k"].shape[2] + ps - 1) // ps * ps
            per_seq = cap_p // ps

            def to_pages(x):
                xp = torch.nn.functional.pad(x, (0, 0, 0, cap_p - x.shape[2]))
                return xp.view(B, cfg.num_kv_heads, per_seq, ps, cfg.head_dim).permute(0, 2, 1, 3, 4).reshape(
                    B * per_seq, cfg.num_kv_heads, ps, cfg.head_dim)
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
                E.eagle_tree_verify_attn_paged(s["q"], kp, vp, table, s["sl"], s["par"], ctx.out, tree_sizes=s["ts"], workspace=ctx.ws,
                                               status=status, num_splits=args.num_splits, events=(e[0], e[1]))
            torch.cuda.synchronize()
            paged[f"page_{ps}"] = {"attn_kernel_ms": statistics.median(e[0].elapsed_time(e[1]) for e in pe[3:]),
                                   "same_bits_as_contiguous": bool(torch.equal(ctx.out.view(torch.int16), ref_bits))}
            del kp, vp
        del ref_bits
        ctx.check()

        # ---- commit of the accepted path for this layer's cache (the step after verification; reported, not part of the
        # headline).  It moves rows in place, so it runs on the last input set, after everything that reads the cache.
        s = ctx.sets[-1]
        ctx.accept(s)
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
        ctx.check()
        commit_ms = c0.elapsed_time(c1) / 50      # back-to-back calls: the larger of kernel time and enqueue time per call
        moved = int(((path >= 0) & (path != torch.arange(T, device=dev, dtype=torch.int32)[None, :])).sum().item())
        commit_bytes = moved * cfg.num_kv_heads * cfg.head_dim * 2 * 2 * 2     # rows that change slot: K and V, read + written
        extras.update({
            "accept_ms": accept_ms, "tokens_per_step": mean_tokens, "accept_rho0": accept_rho0,
            "accept_on_logits": {"ms": accept_logits_ms, "temperature": 1.0,
                                 "sequences_with_the_same_tokens_as_on_probabilities": logits_same, "of": B},
            "tree_expand": {"ms": expand_ms, "rows": B * R_exp, "children": K_exp, "bytes": expand_bytes,
                            "gbs": expand_bytes / (expand_ms * 1e-3) / 1e9, "note": "back-to-back calls on the same rows (warm L2)"},
            "cuda_graph": cuda_graph, "per_layer": per_layer, "fp8_kv": fp8_kv, "paged_attention": paged,
            "kv_commit": {"ms": commit_ms, "rows_moved_per_kv_head": moved, "bytes": commit_bytes,
                          "gbs": commit_bytes / (commit_ms * 1e-3) / 1e9, "bound": "launch + memory latency"}})
    ctx.free()

    # ---- end to end from pinned host buffers, through the library's host-buffer entry point: every step copies all
    # inputs host->device, runs attention + acceptance, and copies the results back
    pinned = dict(q=attn.q, k_cache=attn.k_cache, v_cache=attn.v_cache, seq_lens=attn.seq_lens, tree_sizes=attn.tree_sizes,
                  tree_parent=attn.tree_parent, target_probs=acc.target_probs, draft_probs=acc.draft_probs,
                  draft_tokens=acc.draft_tokens, uniforms=acc.uniforms, greedy=acc.greedy)
    pinned = {k: v.pin_memory() for k, v in pinned.items()}
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
    e2e_value = replicas.whole_job_steps_per_s(e0.elapsed_time(e1), args.e2e_steps, dev)
    # the step driven from host buffers gives the same tokens as the device-resident one (all input sets hold the same data)
    same_tokens = None if args.only_step else bool((runner.bonus_token.numpy() == gpu_bonus).all())
    del runner, pinned
    torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- the other configurations, a few dozen steps each (attention roofline fractions for every shape the target names)
    others = {}
    if not args.only_step and args.other_steps > 0 and args.batch == 0:
        for name in W.CONFIGS:
            if name == cfg.name:
                continue
            o = StepContext(E, W.CONFIGS[name], dev, 0, args.rho, args.num_splits)
            for i in range(5):
                o.step(i)
            torch.cuda.synchronize()
            o.check()
            ms, a_ms, _ = o.timed(args.other_steps, first=5)
            rec = bounds(o, a_ms, pk, False)
            rec.update({"steps": args.other_steps, "ms_per_step": ms / args.other_steps, "steps_per_s": args.other_steps / (ms * 1e-3),
                        "l2": f"rotating over {o.R} input sets" if o.R > 1 else "inputs larger than L2 (single set)"})
            pl = o.per_layer()
            pl["attn_kernel_share_of_layer"] = a_ms / pl["ms_per_layer"]
            rec["per_layer"] = pl
            rec["cuda_graph"] = o.graph_leg()
            rec["fp8_kv"] = o.fp8_leg(a_ms, pk)
            o.check()
            others[name] = rec
            o.free()
            del o
    sampler.stop()

    traffic, traffic_note = ncu_traffic(cfg)
    if head["bound"] == "tensor":
        achieved, peak, roof_unit = head["tflops"], head["tensor_peak"], "TFLOP/s"
    else:     # HBM, or (never for these shapes) the exponentials: reported against the HBM roof
        achieved, peak, roof_unit = head["gbs"], pk["hbm"], "GB/s"
    sm = clocks.get("sm_mhz") if clocks else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": warm,
        "ms_per_step": elapsed_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": B, "num_q_heads": cfg.num_q_heads, "num_kv_heads": cfg.num_kv_heads,
                   "head_dim": cfg.head_dim, "prefix": list(cfg.prefix), "tree": list(cfg.tree), "vocab": cfg.vocab,
                   "greedy": cfg.greedy, "rho": args.rho, "parallelism": f"replicas x{world}",
                   "l2": (f"rotating over {ctx.R} input sets" if ctx.R > 1 else "inputs larger than L2 (single set)")},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
                "api": "eagle_tree_verify_step_host", "same_tokens_as_device_path": same_tokens},
        "roofline": {"bound": "tensor" if head["bound"] == "tensor" else "hbm", "kernel": "split-KV tree attention", "achieved": achieved,
                     "peak": peak, "unit": roof_unit, "frac": achieved / peak, "peak_source": pk["source"] + " (of measured)",
                     "traffic": traffic, "traffic_note": traffic_note, "ms_per_launch": attn_ms,
                     "frac_at_max_clock": (achieved / peak * pk["sm_max_mhz"] / sm) if sm else None, **head},
        "breakdown": {"attn_kernel_ms": attn_ms, "sequence_steps_per_s": value * B, **extras, "workloads": others},
    }
    if not args.no_cpu_baseline and not args.only_step:
        import oracle
        done, secs, cores, kept = oracle_step_sample(attn, acc, args.cpu_budget, keep=True)
        v, share = scaled_steps_per_s(attn, done, secs)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"first {done} of {B} sequences of the same batch (attention + acceptance), {secs:.1f} s, "
                                          f"{share:.3f} of the batch's work; value scaled to whole batches"}
        line["parity"] = parity_record(ctx, gpu_out, gpu_path, gpu_bonus, gpu_alen, kept)
        oracle.set_num_threads(1)
        d1, s1, c1_, _ = oracle_step_sample(attn, acc, min(args.cpu_budget, 6.0))
        oracle.set_num_threads(0)
        v1, share1 = scaled_steps_per_s(attn, d1, s1)
        line["cpu_baseline"]["one_thread"] = {"value": v1, "cores": c1_, "sample": f"first {d1} sequences, {s1:.1f} s, {share1:.3f} of the batch's work"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
