#!/usr/bin/env python
"""Benchmark of the LCA prefill hot path (condense + condensed attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config mla_128k] [--impl ours|reference]

One "step" = one pass of the whole hot path over one synthetic sequence of the chosen
configuration: lca_condense (summary query, group scores, softmax, pooling, anchors, local
window) followed by lca_prefill_attention.  Inputs are resident in HBM for `value`; the `e2e`
figure repeats the step from pinned host buffers with the host<->device copies inside the timed
region.  With N > 1 every rank runs an independent replica (the path has no exchange step):
value = N * tokens / max-over-ranks time.

--impl reference times the CPU oracle (fp64, OpenMP) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2604_12452_b200 import inputs as I

METRIC = "lca_prefill_tokens_per_s"
UNIT = "tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum of attn_tc2_kernel at mla_32k (L=32768, H=16) divided by
# L*H: the kernel reads every query row and writes every output row once, the key/value stream stays in L2.
ATTN_DRAM_BYTES_PER_TOKEN_HEAD = (642.586880e6 + 497.310208e6) / (32768 * 16)


# ---------------------------------------------------------------------------- work counts
def key_visits(L: int, g: int, w: int) -> int:
    """sum over query positions of (representatives + local tokens) it attends to."""
    t = np.arange(1, L + 1, dtype=np.int64)
    mt = np.where(t < w + g, 0, (t - w) // g)
    return int((mt + (t - mt * g)).sum())


def attention_flops(cfg) -> float:
    dk = cfg.d_sem + cfg.d_pos if cfg.variant == "mla" else cfg.d_sem
    return float(key_visits(cfg.seq_len, cfg.group_size, cfg.window)) * cfg.n_q_heads * 2.0 * (dk + cfg.d_sem) * cfg.batch


def condense_bytes(cfg) -> float:
    """Algorithmic HBM bytes of lca_condense: history rows read once, query tail read once,
    representatives + anchors written, local window read and written."""
    L, g, w = cfg.seq_len, cfg.group_size, cfg.window
    m = 0 if L < w + g else (L - w) // g
    k = L - m * g
    d_pos = cfg.d_pos if cfg.variant == "mla" else cfg.d_sem
    row = (cfg.d_sem + d_pos) * 2 * cfg.n_kv_heads
    qrow = ((cfg.d_sem + cfg.d_pos) if cfg.variant == "mla" else cfg.d_sem) * 2 * cfg.n_q_heads
    return float(cfg.batch) * (m * g * row + min(g, L) * qrow + m * row + 4 * m * cfg.n_kv_heads + 2 * k * row)


def max_over_ranks(ms: float, dist, device) -> float:
    """The time of a multi-rank step is the slowest rank's (replicas run independently)."""
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """tokens/s over all ranks: every rank processes its own sequence in the same wall time."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], tflops_burst=d["bf16_tflops"], tflops_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


# ---------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------- CPU oracle
def sample_rows(cfg, n_rows: int, seed: int = 0):
    from oracle import parity as P
    return P.sample_positions(cfg.seq_len, cfg.group_size, cfg.window, n_uniform=max(0, n_rows - 18), seed=seed)[:max(n_rows, 1)]


def oracle_sample(cfg, small, n_rows: int, n_heads: int, seed: int = 0):
    """Time the oracle on a bounded sample: condensation of the whole sequence plus `n_rows` stratified query
    rows x `n_heads` heads.  Returns (tokens_per_s_estimate, description, threads, oracle results)."""
    from oracle import lca_oracle as O, parity as P
    L, g, w, H = cfg.seq_len, cfg.group_size, cfg.window, cfg.n_q_heads
    rows = sample_rows(cfg, n_rows, seed)
    heads = np.arange(min(n_heads, H))
    t0 = time.perf_counter()
    full = P.mla_pipeline(small["ckv"], small["kr"], small["q_sem"], small["q_pos"], g, w, cfg.softmax_scale)
    t_cond = time.perf_counter() - t0                    # summary query + condensation of the whole sequence
    m = full["cond"]["m"]
    rep_sem = O.bits_to_f64(full["cond"]["cache_sem_bits"][:m]) if m else None
    rep_pos = O.bits_to_f64(full["cond"]["cache_pos_bits"][:m]) if m else None
    ckv64, kr64 = O.torch_bf16_to_f64(small["ckv"]), O.torch_bf16_to_f64(small["kr"])
    qs = O.torch_bf16_to_f64(small["q_sem_rows"][:len(rows)][:, heads])
    qp = O.torch_bf16_to_f64(small["q_pos_rows"][:len(rows)][:, heads])
    t0 = time.perf_counter()
    out, lse = O.mla_prefill_rows(qs, qp, rows, ckv64, kr64, rep_sem, rep_pos, g, w, P.f32(cfg.softmax_scale))
    t_rows = time.perf_counter() - t0
    full.update(rows=rows, out=out, lse=lse)
    mt = np.where(rows + 1 < w + g, 0, (rows + 1 - w) // g)
    sampled_visits = float((mt + (rows + 1 - mt * g)).sum()) * len(heads)
    total_visits = float(key_visits(L, g, w)) * H
    est_total = t_cond + t_rows * total_visits / max(sampled_visits, 1.0)
    desc = (f"condense of all {L} tokens ({t_cond:.2f}s) + {len(rows)} stratified query rows x {len(heads)} of {H} heads "
            f"({t_rows:.2f}s), scaled by visited (query,key,head) triples {sampled_visits:.3g}/{total_visits:.3g}")
    full.update(heads=heads)
    return L * cfg.batch / est_total, desc, O.num_threads(), full


def gather_oracle_inputs(cfg, inp, n_rows, seed=0):
    """CPU copies of what the oracle sample needs (the K/V streams and the sampled query rows)."""
    L, g = cfg.seq_len, cfg.group_size
    rows = sample_rows(cfg, n_rows, seed)
    if inp is None:
        # no GPU and queries too large for host memory (timing only, nothing is compared): the keys / values of the whole
        # sequence, the query tail, and as many further query rows as are sampled, drawn for the positions before the tail
        n = len(rows)
        part = I.make_mla_inputs(cfg, "cpu", q_positions=slice(L - g - n, L))
        return dict(ckv=part["ckv"], kr=part["kr"], q_sem=part["q_sem"][n:], q_pos=part["q_pos"][n:],
                    q_sem_rows=part["q_sem"][:n], q_pos_rows=part["q_pos"][:n])
    idx = torch.from_numpy(rows).to(inp["q_sem"].device)
    return dict(ckv=inp["ckv"].cpu(), kr=inp["kr"].cpu(), q_sem=inp["q_sem"][L - g:].cpu(), q_pos=inp["q_pos"][L - g:].cpu(),
                q_sem_rows=inp["q_sem"][idx].cpu(), q_pos_rows=inp["q_pos"][idx].cpu())


def parity_record(ref, out_rows, cache=None, kind="mla"):
    """Raw comparison figures of a device result with the oracle's (by-product of the oracle leg): attention
    output on the sampled rows, and the condensed cache in full when given."""
    from oracle import lca_oracle as O, parity as P
    vmax = ref["vmax"][None]
    ro = ref["out"]
    st = P.output_stats(out_rows, ro, vmax)
    rec = dict(rows=int(ro.shape[0]), heads=int(ro.shape[1]), max_abs=st["max_abs"], mean_abs=st["mean_abs"], max_ref=st["max_ref"],
               mean_ref=st["mean_ref"], n_above_2e2=st["n_above_2e2"], max_abs_unit_scale=st["max_abs_unit_scale"],
               worst_over_derived_bound=st["worst_over_bound"])
    if cache is not None:
        cs = P.condense_stats(O.torch_bf16_to_bits(cache["cache_sem"]), O.torch_bf16_to_bits(cache["cache_pos"]),
                              cache["anchor_idx"].cpu().numpy(), ref["cond"], kind)
        rec.update(anchor_mismatches=cs["anchor_mismatches"], near_tie_groups=cs["near_tie_groups"], groups=cs["m"],
                   copied_rows_differing=cs["pos_rows_differ"] + cs["local_sem_rows_differ"],
                   crep_off_by_one_ulp=cs["crep_off_by_one_ulp"], crep_beyond_one_ulp=cs["crep_bad"], crep_elems=cs["crep_elems"])
    return rec


# -------------------------------------------------------------------------------- main arms
def run_reference(args, cfg, rank, world):
    if rank != 0:
        return
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    inp = I.make_mla_inputs(cfg, dev) if cfg.seq_len * cfg.n_q_heads * 576 * 2 < 8e9 or dev != "cpu" else None
    small = gather_oracle_inputs(cfg, inp, args.ref_rows)
    del inp
    times, vals = [], []
    desc, threads = "", 1
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        v, desc, threads, _ = oracle_sample(cfg, small, args.ref_rows, args.ref_heads)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
            vals.append(v)
    value = float(np.mean(vals))
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * cfg.seq_len * cfg.batch / value, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(cfg, args.gpus),
                cpu_baseline=dict(value=value, unit=UNIT, cores=threads, kind="oracle", sample=desc),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                sample_wall_s=float(np.mean(times)))
    print(json.dumps(line))


L2_BYTES = 126 << 20


def step_bytes(cfg):
    """Bytes one step reads and writes in HBM: queries, keys / values, output."""
    d_qk = cfg.d_sem + cfg.d_pos                          # MLA: latent + rope; GQA: head dimension (d_pos = 0)
    n_kv = 1 if cfg.variant == "mla" else 2 * cfg.n_kv_heads      # MLA: one shared [c | k_R] row; GQA: K and V per KV head
    return 2 * cfg.batch * cfg.seq_len * (cfg.n_q_heads * (d_qk + cfg.d_sem) + n_kv * d_qk)


def needs_l2_flush(cfg):
    return step_bytes(cfg) < 2 * L2_BYTES


def workload_config(cfg, n_gpus):
    return dict(workload=f"{cfg.name}: one {cfg.variant.upper()} layer, batch {cfg.batch}, L={cfg.seq_len}, "
                         f"H={cfg.n_q_heads}, d_sem={cfg.d_sem}, d_pos={cfg.d_pos}, g={cfg.group_size}, w={cfg.window}, causal",
                seq_len=cfg.seq_len, n_q_heads=cfg.n_q_heads, group_size=cfg.group_size, window=cfg.window,
                parallelism=f"replicas x{n_gpus}" if n_gpus > 1 else "single GPU",
                l2_policy=("a 256 MB buffer is written between timed steps (the step's tensors would fit the 126 MB L2)"
                           if needs_l2_flush(cfg) else
                           f"inputs and outputs of a step ({step_bytes(cfg) / 1e9:.1f} GB) exceed the 126 MB L2; no flush needed"))


def run_ours(args, cfg, rank, world, local_rank):
    from paper_2604_12452_b200 import build
    build.build()
    from paper_2604_12452_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    L, g = cfg.seq_len, cfg.group_size
    inp = I.make_mla_inputs(cfg, dev)
    p = B.params_from_config(cfg, batch=1)
    m, k = B.lca_partition(p)
    out = torch.empty((1, L, cfg.n_q_heads, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    cache = dict(cache_sem=torch.empty((1, m + k, 1, cfg.d_sem), dtype=torch.bfloat16, device=dev),
                 cache_pos=torch.empty((1, m + k, 1, cfg.d_pos), dtype=torch.bfloat16, device=dev),
                 anchor_idx=torch.empty((1, max(m, 1), 1), dtype=torch.int32, device=dev))
    ws_c = B.workspace(p, B.LCA_WS_CONDENSE, dev)
    ws_a = B.workspace(p, B.LCA_WS_PREFILL, dev)
    q_tail_sem, q_tail_pos = inp["q_sem"][L - g:], inp["q_pos"][L - g:]

    def step(ev=None):
        if ev:
            ev[0].record()
        B.condense(p, q_tail_sem, q_tail_pos, inp["ckv"], inp["kr"], out=cache, ws=ws_c)
        if ev:
            ev[1].record()
        B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cache["cache_sem"],
                            cache["cache_pos"], out=out, ws=ws_a)
        if ev:
            ev[2].record()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    launches0 = B.lca_launch_count()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if needs_l2_flush(cfg) else None
    barrier()
    for i in range(args.steps):
        if flush is not None:
            flush.zero_()                          # evicts the step's tensors from L2; outside the timed events
        step(evs[i])
    barrier()
    launches = B.lca_launch_count() - launches0
    clocks = sampler.stop()
    if flush is not None:
        total_ms = float(sum(e[0].elapsed_time(e[2]) for e in evs))      # the flushes lie between the steps
    else:
        total_ms = evs[0][0].elapsed_time(evs[-1][2])
    t_cond = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    t_attn = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    status = B.lca_last_device_status()
    if status != 0:
        raise RuntimeError(f"device status {status}: {B.lca_status_string(status)}")
    total_ms = max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / args.steps
    value = whole_job_value(L * cfg.batch, world, ms_per_step)

    # ---- end to end: pinned host buffers; every step copies its inputs host -> device, runs the two
    # entry points and copies its output device -> host.  Up to three streams with their own device
    # buffers take the steps in turn, so the upload of one step overlaps the kernels of the previous
    # one and the download of the one before (PCIe is full duplex); the timed region covers all
    # copies of all steps.
    e2e = None
    if not args.no_e2e:
        try:
            host = {kname: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for kname, v in inp.items()}
            n_e2e = max(2, args.e2e_steps)
            h2d = sum(v.numel() * v.element_size() for v in host.values())
            d2h = out.numel() * out.element_size()
            per_set = h2d + d2h + sum(v.numel() * v.element_size() for v in cache.values() if torch.is_tensor(v))
            free_bytes = torch.cuda.mem_get_info(dev)[0]
            # a third set costs another pinned output buffer per rank: only where few ranks share the host
            n_sets = 3 if (free_bytes > 2 * per_set + (8 << 30) and world <= 2) else 2
            sets = []
            for i in range(n_sets):
                dev_in = inp if i == 0 else {kname: torch.empty_like(v) for kname, v in inp.items()}
                sets.append(dict(
                    stream=torch.cuda.Stream(), inp=dev_in, out=out if i == 0 else torch.empty_like(out),
                    cache=cache if i == 0 else {kname: torch.empty_like(v) for kname, v in cache.items()},
                    ws_c=ws_c if i == 0 else torch.empty_like(ws_c), ws_a=ws_a if i == 0 else torch.empty_like(ws_a),
                    host_out=torch.empty(out.shape, dtype=out.dtype, pin_memory=True)))

            def e2e_step(st):
                with torch.cuda.stream(st["stream"]):
                    for kname in st["inp"]:
                        st["inp"][kname].copy_(host[kname], non_blocking=True)
                    B.condense(p, st["inp"]["q_sem"][L - g:], st["inp"]["q_pos"][L - g:], st["inp"]["ckv"], st["inp"]["kr"],
                               out=st["cache"], ws=st["ws_c"])
                    B.prefill_attention(p, st["inp"]["q_sem"], st["inp"]["q_pos"], st["inp"]["ckv"], st["inp"]["kr"],
                                        st["cache"]["cache_sem"], st["cache"]["cache_pos"], out=st["out"], ws=st["ws_a"])
                    st["host_out"].copy_(st["out"], non_blocking=True)

            barrier()
            for st in sets:
                st["stream"].wait_stream(torch.cuda.current_stream())
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for st in sets:
                st["stream"].wait_event(e0)
            for i in range(n_e2e):
                e2e_step(sets[i % n_sets])
            for st in sets:
                torch.cuda.current_stream().wait_stream(st["stream"])
            e1.record()
            barrier()
            t_e2e = max_over_ranks(e0.elapsed_time(e1) / n_e2e, dist, dev)
            e2e = dict(value=whole_job_value(L * cfg.batch, world, t_e2e), unit=UNIT, h2d_bytes_per_step=h2d,
                       d2h_bytes_per_step=d2h, steps=n_e2e, ms_per_step=t_e2e,
                       note=f"{n_sets} streams take the steps in turn: uploads overlap the kernels and the downloads of earlier steps")
            del host, sets
            torch.cuda.empty_cache()
        except RuntimeError as ex:      # e.g. not enough pinnable host memory on this machine
            e2e = dict(value=None, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0, error=str(ex)[:200])

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    want_oracle = not args.no_cpu_baseline
    flops = attention_flops(cfg)
    tfl = flops / (t_attn * 1e-3) / 1e12
    cbytes = condense_bytes(cfg)
    cgbs = cbytes / (t_cond * 1e-3) / 1e9
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic", config=workload_config(cfg, world), clocks=clocks, gpu_launches=int(launches),
                e2e=e2e,
                roofline=dict(bound="tensor", achieved=tfl, peak=peaks["tflops_sustained"], unit="TFLOP/s",
                              frac=tfl / peaks["tflops_sustained"],
                              traffic=ATTN_DRAM_BYTES_PER_TOKEN_HEAD * L * cfg.n_q_heads if cfg.variant == "mla" else None,
                              traffic_note="dram read+write of one ncu capture at mla_32k (profiles/), scaled by tokens x heads",
                              kernel="lca_prefill_attention", flops_per_launch=flops, ms_per_launch=t_attn,
                              peak_kind=f"{peaks['source']} cuBLAS bf16, sustained (kernel timed inside a long step)",
                              frac_of_burst=tfl / peaks["tflops_burst"], frac_of_nominal_2250=tfl / 2250.0),
                roofline_condense=dict(bound="hbm", achieved=cgbs, peak=peaks["hbm_gbs"], unit="GB/s",
                                       frac=cgbs / peaks["hbm_gbs"], traffic=None, kernel="lca_condense (all launches)",
                                       bytes_per_launch=cbytes, ms_per_launch=t_cond, peak_kind=f"{peaks['source']} copy"),
                attention_impl=args.attn_impl)
    parity = {}
    if want_oracle:
        small = gather_oracle_inputs(cfg, inp, args.ref_rows)
        v, desc, threads, ref = oracle_sample(cfg, small, args.ref_rows, args.ref_heads)
        line["cpu_baseline"] = dict(value=v, unit=UNIT, cores=threads, kind="oracle", sample=desc)
        idx = torch.from_numpy(ref["rows"]).to(dev)
        hd = torch.from_numpy(ref["heads"]).to(dev)
        parity[cfg.name] = parity_record(ref, out[0][idx][:, hd], {kk: cache[kk][0] for kk in cache})
        del small, ref
    extras = {}
    if not args.no_extras and world == 1:
        side = [("dense_mla_at_this_config", lambda: measure_dense_here(B, dev, cfg, inp, out, t_cond + t_attn)),
                ("value_projection", lambda: measure_value_projection(B, dev, cfg, out, peaks))]
        for name, fn in side:
            try:
                extras[name] = fn()
            except Exception as ex:        # report, never lose the main line
                extras[name] = dict(error=str(ex)[:200])
        del inp, out, cache
        torch.cuda.empty_cache()
        side = [("config1", lambda: measure_mla_small(B, dev, "mla_1k", want_oracle, parity)),
                ("config2", lambda: measure_mla_small(B, dev, "mla_32k", want_oracle, parity)),
                ("decode_config", lambda: measure_decode_config(B, dev, args.decode_batch, peaks, parity=parity if want_oracle else None)),
                ("gqa_config", lambda: measure_gqa_config(B, dev, peaks, parity=parity if want_oracle else None)),
                ("dense_mla_comparison", lambda: measure_dense_comparison(B, dev, peaks)),
                ("scaling", lambda: measure_scaling(B, dev, peaks))]
        for name, fn in side:
            try:
                extras[name] = fn()
            except Exception as ex:
                extras[name] = dict(error=str(ex)[:200])
            torch.cuda.empty_cache()
    if parity:
        extras["parity"] = dict(note="device results against the fp64 oracle on the same bits, raw figures: |err| of the attention output "
                                     "on sampled rows (max_abs_unit_scale: elements with |ref| <= 1.5 in columns without a x4 needle; "
                                     "worst_over_derived_bound: against max(2e-2, 2^-9 (vmax_c + |ref|) + 2^-8 |ref|)), anchors and copied "
                                     "rows of the whole condensed cache (bit-exact: mismatches must be 0; near_tie_groups counts groups whose "
                                     "two best fp64 scores lie within 1e-6 relative), c_rep elements one bf16 ulp off",
                                **parity)
    line["extras"] = extras
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def time_cuda(fn, warmup=3, iters=5):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def time_cuda_graph(fn, n=10):
    """Device time per call of a short sequence of launches: n calls captured into one CUDA graph, replayed twice
    (eager calls of a few microseconds each measure the host's launch rate instead)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(n):
                fn()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        graph.replay()
        graph.replay()
        e1.record(side)
        torch.cuda.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    return e0.elapsed_time(e1) / (2 * n)


def measure_decode_config(B, dev, batch, peaks, warmup=3, iters=5, parity=None):
    """Config 4: lca_condense over `batch` contexts of 65536 tokens (the HBM-bound figure), then
    lca_decode_attention of one new query per sequence over the condensed cache."""
    cfg = I.scaled(I.CONFIGS["mla_decode"], batch=batch)
    L, g, H = cfg.seq_len, cfg.group_size, cfg.n_q_heads
    ckv = torch.empty((batch, L, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    kr = torch.empty((batch, L, cfg.d_pos), dtype=torch.bfloat16, device=dev)
    q_tail_sem = torch.empty((batch, g, H, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    q_tail_pos = torch.empty((batch, g, H, cfg.d_pos), dtype=torch.bfloat16, device=dev)
    for b in range(batch):
        one = I.make_mla_inputs(cfg, dev, batch_index=b, q_positions=slice(L - g, L))
        ckv[b], kr[b], q_tail_sem[b], q_tail_pos[b] = one["ckv"], one["kr"], one["q_sem"], one["q_pos"]
    p = B.params_from_config(cfg, batch=batch)
    m, k = B.lca_partition(p)
    cap = m + k + 1                                   # + the new token's own row
    cache = dict(cache_sem=torch.zeros((batch, m + k, 1, cfg.d_sem), dtype=torch.bfloat16, device=dev),
                 cache_pos=torch.zeros((batch, m + k, 1, cfg.d_pos), dtype=torch.bfloat16, device=dev),
                 anchor_idx=torch.empty((batch, m, 1), dtype=torch.int32, device=dev))
    ws = B.workspace(p, B.LCA_WS_CONDENSE, dev)
    t_cond = time_cuda(lambda: B.condense(p, q_tail_sem, q_tail_pos, ckv, kr, out=cache, ws=ws), warmup, iters)
    cfg_b = I.scaled(cfg, batch=batch)
    cbytes = condense_bytes(cfg_b)
    # decode: cache with one appended row per sequence
    dsem = torch.zeros((batch, cap, 1, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    dpos = torch.zeros((batch, cap, 1, cfg.d_pos), dtype=torch.bfloat16, device=dev)
    dsem[:, :m + k] = cache["cache_sem"]
    dpos[:, :m + k] = cache["cache_pos"]
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed + 99)
    dsem[:, m + k] = torch.randn((batch, 1, cfg.d_sem), generator=gen, device=dev).bfloat16()
    dpos[:, m + k] = torch.randn((batch, 1, cfg.d_pos), generator=gen, device=dev).bfloat16()
    q_new_sem = torch.randn((batch, H, cfg.d_sem), generator=gen, device=dev).bfloat16()
    q_new_pos = torch.randn((batch, H, cfg.d_pos), generator=gen, device=dev).bfloat16()
    rows = torch.full((batch,), cap, dtype=torch.int32, device=dev)
    out = torch.empty((batch, H, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    wsd = B.workspace(p, B.LCA_WS_DECODE, dev)
    t_dec = time_cuda(lambda: B.decode_attention(p, q_new_sem, q_new_pos, dsem, dpos, rows, m, out=out, ws=wsd), warmup, iters)
    # online cache update (Sec. 4.3) at the moment every sequence has w + g buffered tokens
    upd = None
    try:
        cap_u = m + cfg.window + g
        usem = torch.randn((batch, cap_u, 1, cfg.d_sem), generator=gen, device=dev).bfloat16()
        upos = torch.randn((batch, cap_u, 1, cfg.d_pos), generator=gen, device=dev).bfloat16()
        wsu = B.workspace(p, B.LCA_WS_UPDATE, dev)
        times = []
        for _ in range(3):
            n_rep_t = torch.full((batch,), m, dtype=torch.int32, device=dev)
            rows_t = torch.full((batch,), cap_u, dtype=torch.int32, device=dev)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.decode_update(p, q_tail_sem, q_tail_pos, usem, upos, n_rep_t, rows_t, ws=wsu)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        upd = dict(us_per_update_all_sequences=min(times) * 1e3, amortised_us_per_token=min(times) * 1e3 / g,
                   note="every g-th decode step: summary query, condense the earliest g buffered tokens, move the window up")
        del usem, upos
        # the same moment on the ring layout (token n at row n % (w + g), representatives behind the ring): nothing
        # moves; timed with the query tails and with a summary query the caller kept up to date while decoding
        R = cfg.window + g
        cap_r = R + m + 8
        rsem = torch.randn((batch, cap_r, 1, cfg.d_sem), generator=gen, device=dev).bfloat16()
        rpos = torch.randn((batch, cap_r, 1, cfg.d_pos), generator=gen, device=dev).bfloat16()
        qbar_ready = torch.randn((batch, 1, cfg.d_sem + cfg.d_pos), generator=gen, device=dev, dtype=torch.float32)
        n_tok_full = torch.full((batch,), m * g + R, dtype=torch.int32, device=dev)
        ring = {}
        for name, qb in (("tails", None), ("ready_summary_query", qbar_ready)):
            times = []
            for _ in range(3):
                n_rep_t = torch.full((batch,), m, dtype=torch.int32, device=dev)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                B.decode_update_ring(p, q_tail_sem, q_tail_pos, rsem, rpos, n_rep_t, n_tok_full, qbar=qb, ws=wsu)
                e1.record()
                torch.cuda.synchronize()
                times.append(e0.elapsed_time(e1))
                assert int(n_rep_t.min()) == m + 1
            ring[name] = min(times) * 1e3
        # decode over the ring one token after that update: g - 1 stale rows inside the ring are masked out
        n_rep_t = torch.full((batch,), m + 1, dtype=torch.int32, device=dev)
        n_tok_t = torch.full((batch,), m * g + R + 1, dtype=torch.int32, device=dev)
        out_r = torch.empty_like(out)
        t_ring_dec = time_cuda(lambda: B.decode_attention_ring(p, q_new_sem, q_new_pos, rsem, rpos, n_rep_t, n_tok_t, out=out_r, ws=wsd),
                               warmup, iters)
        # one call per decode step with a running summary query: a step in which no sequence is due, and one in which all are
        qsum = torch.zeros((batch, 1, cfg.d_sem + cfg.d_pos), dtype=torch.float64, device=dev)
        qcount = torch.zeros((batch,), dtype=torch.int32, device=dev)
        anc = torch.empty((batch, 1), dtype=torch.int32, device=dev)
        n_rep_idle = torch.full((batch,), m, dtype=torch.int32, device=dev)
        n_tok_idle = torch.full((batch,), m * g + R - 1, dtype=torch.int32, device=dev)
        t_step_idle = time_cuda_graph(lambda: B.decode_step_update_ring(p, q_new_sem, q_new_pos, qsum, qcount, rsem, rpos, n_rep_idle,
                                                                        n_tok_idle, ws=wsu, anchor=anc))
        n_rep_t = torch.full((batch,), m, dtype=torch.int32, device=dev)

        def due_step():
            n_rep_t.fill_(m)                                       # every sequence is due again (a 64-element fill)
            B.decode_step_update_ring(p, q_new_sem, q_new_pos, qsum, qcount, rsem, rpos, n_rep_t, n_tok_full, ws=wsu, anchor=anc)
        t_step_due = time_cuda_graph(due_step)
        assert int(n_rep_t.min()) == m + 1 and int(qcount.max()) == 0 and int(anc.min()) >= 0
        upd["ring_layout"] = dict(us_per_update_all_sequences=ring["tails"], us_with_ready_summary_query=ring["ready_summary_query"],
                                  amortised_us_per_token_from_tails=ring["tails"] / g,
                                  decode_us=t_ring_dec * 1e3, step_update_us_nobody_due=t_step_idle * 1e3,
                                  step_update_us_all_due=t_step_due * 1e3,
                                  step_update_amortised_us_per_token=(t_step_idle * (g - 1) + t_step_due) * 1e3 / g,
                                  note="lca_decode_update_ring / lca_decode_attention_ring: one new row per sequence, no row moves; "
                                       "step_update = lca_decode_step_update_ring, called at every decode step (running summary query), device time "
                                       "from a CUDA graph of ten calls; its amortised figure = (g - 1) steps with nobody due + one with all due")
        del rsem, rpos
    except Exception as ex:
        upd = dict(error=str(ex)[:200])
    # the decode launch repeated for about a second: the clock then sits at what the power cap allows (as in the main
    # benchmark); taken last, so that the burst figures above are not measured on a GPU that is already at the cap
    t_dec_sustained = time_cuda(lambda: B.decode_attention(p, q_new_sem, q_new_pos, dsem, dpos, rows, m, out=out, ws=wsd), 0, 10000) \
        if batch >= 32 else None
    if parity is not None:
        # oracle on the first and the last sequence: the whole condensed cache and the decode output of every head
        from oracle import lca_oracle as O, parity as P
        recs = []
        for b in sorted({0, batch - 1}):
            ref = P.mla_pipeline(ckv[b].cpu(), kr[b].cpu(), q_tail_sem[b].cpu(), q_tail_pos[b].cpu(), g, cfg.window, cfg.softmax_scale)
            ro, _ = O.mla_decode(O.torch_bf16_to_f64(q_new_sem[b].cpu()), O.torch_bf16_to_f64(q_new_pos[b].cpu()),
                                 O.torch_bf16_to_f64(dsem[b, :, 0].cpu()), O.torch_bf16_to_f64(dpos[b, :, 0].cpu()), m, P.f32(cfg.softmax_scale))
            ref.update(out=ro[None])
            recs.append(parity_record(ref, out[b][None], {kk: cache[kk][b] for kk in cache}))
        parity["mla_decode"] = dict(sequences=sorted({0, batch - 1}), per_sequence=recs)
    flops = float(batch) * H * cap * 2.0 * (cfg.d_sem + cfg.d_pos + cfg.d_sem)
    kv_bytes = float(batch) * cap * (cfg.d_sem + cfg.d_pos) * 2
    full_bytes = float(batch) * (L + 1) * (cfg.d_sem + cfg.d_pos) * 2
    return dict(workload=f"mla_decode: batch {batch}, contexts of {L} tokens, H={H}, g={g}, w={cfg.window}",
                condense=dict(ms=t_cond, bytes=cbytes, gbs=cbytes / t_cond / 1e6, frac_of_measured_hbm=cbytes / t_cond / 1e6 / peaks["hbm_gbs"]),
                decode=dict(us=t_dec * 1e3, us_note=f"{iters} launches after {warmup} warm-up launches (a burst: the clock has not yet settled at the power cap)",
                            us_sustained=None if t_dec_sustained is None else t_dec_sustained * 1e3,
                            us_sustained_note="10000 launches back to back (about a second): SM clock at the power cap",
                            rows_per_seq=cap, tflops=flops / t_dec / 1e9, kv_gbs=kv_bytes / t_dec / 1e6,
                            kv_bytes_condensed=kv_bytes, kv_bytes_full_mla=full_bytes, kv_reduction=1.0 - kv_bytes / full_bytes),
                online_update=upd)


def measure_gqa_config(B, dev, peaks, warmup=3, iters=5, seq_len=None, parity=None):
    """Config 5: GQA variant (pool V, select K per KV head): condense + prefill attention.
    `seq_len` shortens the sequence (profiler captures of the same kernels on a small case)."""
    cfg = I.CONFIGS["gqa_64k"] if not seq_len else I.scaled(I.CONFIGS["gqa_64k"], seq_len=seq_len)
    L, g = cfg.seq_len, cfg.group_size
    inp = I.make_gqa_inputs(cfg, dev)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, None, inp["q"][L - g:], inp["v"], inp["k"])
    out = torch.empty((1, L, cfg.n_q_heads, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    ws = B.workspace(p, B.LCA_WS_CONDENSE, dev)
    t_cond = time_cuda(lambda: B.condense(p, None, inp["q"][L - g:], inp["v"], inp["k"], out=cond, ws=ws), warmup, iters)
    t_attn = time_cuda(lambda: B.prefill_attention(p, None, inp["q"], inp["v"], inp["k"], cond["cache_sem"], cond["cache_pos"], out=out),
                       warmup, iters)
    if parity is not None:
        from oracle import parity as P
        rows = P.sample_positions(L, g, cfg.window, n_uniform=14, seed=5)
        idx = torch.from_numpy(rows).to(dev)
        ref = P.gqa_pipeline(inp["q"][L - g:].cpu(), inp["k"].cpu(), inp["v"].cpu(), g, cfg.window, cfg.softmax_scale, inp["q"][idx].cpu(), rows)
        parity[cfg.name] = parity_record(ref, out[0][idx], {kk: cond[kk][0] for kk in ("cache_sem", "cache_pos", "anchor_idx")}, kind="gqa")
    flops = attention_flops(cfg)
    cbytes = condense_bytes(cfg)
    res = dict(workload=f"gqa_64k: L={L}, {cfg.n_q_heads} q heads / {cfg.n_kv_heads} kv heads, d={cfg.d_sem}, g={g}, w={cfg.window}",
               tokens_per_s=L / ((t_cond + t_attn) * 1e-3), condense_ms=t_cond, condense_gbs=cbytes / t_cond / 1e6,
               attention_ms=t_attn, attention_tflops=flops / t_attn / 1e9,
               attention_frac_of_measured_burst=flops / t_attn / 1e9 / peaks["tflops_burst"])
    if not seq_len:
        # decode over condensed caches of this shape: 64 sequences, one new query each (HBM-bound: K and V of every row once)
        m, k = B.lca_partition(p)
        nb, cap = 64, m + k + 1
        gen = torch.Generator(device=dev)
        gen.manual_seed(cfg.seed + 7)
        ck = torch.randn((nb, cap, cfg.n_kv_heads, cfg.d_sem), generator=gen, device=dev).bfloat16()
        cv = torch.randn((nb, cap, cfg.n_kv_heads, cfg.d_sem), generator=gen, device=dev).bfloat16()
        qn = torch.randn((nb, cfg.n_q_heads, cfg.d_sem), generator=gen, device=dev).bfloat16()
        pd = B.params_from_config(cfg, batch=nb)
        rows_t = torch.full((nb,), cap, dtype=torch.int32, device=dev)
        od = torch.empty((nb, cfg.n_q_heads, cfg.d_sem), dtype=torch.bfloat16, device=dev)
        wsd = B.workspace(pd, B.LCA_WS_DECODE, dev)
        t_dec = time_cuda(lambda: B.decode_attention(pd, None, qn, cv, ck, rows_t, m, out=od, ws=wsd), warmup, iters)
        kv_bytes = float(nb) * cap * cfg.n_kv_heads * cfg.d_sem * 2 * 2
        res["decode"] = dict(batch=nb, rows_per_seq=cap, us=t_dec * 1e3, kv_gbs=kv_bytes / t_dec / 1e6,
                             frac_of_measured_hbm=kv_bytes / t_dec / 1e6 / peaks["hbm_gbs"])
    return res


def measure_mla_small(B, dev, name, want_oracle, parity):
    """Configs 1 and 2: the same step (condense + prefill attention) on the smaller MLA configurations, with an L2
    flush between repetitions; the oracle on every row (config 1) or on sampled rows (config 2)."""
    cfg = I.CONFIGS[name]
    L, g = cfg.seq_len, cfg.group_size
    inp = I.make_mla_inputs(cfg, dev)
    p = B.params_from_config(cfg, batch=1)
    cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
    out = torch.empty((1, L, cfg.n_q_heads, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    ws_c, ws_a = B.workspace(p, B.LCA_WS_CONDENSE, dev), B.workspace(p, B.LCA_WS_PREFILL, dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    times = []
    for i in range(8):
        flush.zero_()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"], out=cond, ws=ws_c)
        e[1].record()
        B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"], cond["cache_pos"], out=out, ws=ws_a)
        e[2].record()
        torch.cuda.synchronize()
        if i >= 3:
            times.append((e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])))
    t_c, t_a = float(np.mean([t[0] for t in times])), float(np.mean([t[1] for t in times]))
    if want_oracle:
        from oracle import parity as P
        rows = np.arange(L) if L <= 2048 else P.sample_positions(L, g, cfg.window, n_uniform=14, seed=3)
        idx = torch.from_numpy(rows).to(dev)
        ref = P.mla_pipeline(inp["ckv"].cpu(), inp["kr"].cpu(), inp["q_sem"][L - g:].cpu(), inp["q_pos"][L - g:].cpu(), g, cfg.window,
                             cfg.softmax_scale, inp["q_sem"][idx].cpu(), inp["q_pos"][idx].cpu(), rows)
        parity[name] = parity_record(ref, out[0][idx], {kk: cond[kk][0] for kk in ("cache_sem", "cache_pos", "anchor_idx")})
    fl = attention_flops(cfg)
    return dict(workload=workload_config(cfg, 1)["workload"], tokens_per_s=L / ((t_c + t_a) * 1e-3), condense_us=t_c * 1e3,
                attention_us=t_a * 1e3, attention_tflops=fl / t_a / 1e9, condense_gbs=condense_bytes(cfg) / t_c / 1e6,
                l2_policy="a 256 MB buffer is written between repetitions")


def measure_dense_here(B, dev, cfg, inp, out, t_lca_ms):
    """Dense absorbed-MLA attention (Eq. 5: window >= L) on the benchmark's own tensors, one repetition (it is an
    O(L^2) launch of seconds), beside the LCA step measured above."""
    L, g = cfg.seq_len, cfg.group_size
    cd = I.scaled(cfg, window=L)
    p = B.params_from_config(cd, batch=1)
    cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
    t = time_cuda(lambda: B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"],
                                              cond["cache_pos"], out=out), 0, 1)
    fl = attention_flops(cd)
    return dict(workload=f"{cfg.name} with window = L (no condensation)", dense_ms=t, dense_flops=fl, dense_tflops=fl / t / 1e9,
                lca_step_ms=t_lca_ms, speedup_lca_over_dense=t / t_lca_ms,
                note="run after the LCA measurements: it overwrites the output buffer")


def measure_value_projection(B, dev, cfg, out, peaks):
    """out_v = attn_latent . W^UV on the benchmark's latent output (Alg. 1: v = c W^UV): HBM-bound by arithmetic."""
    H = cfg.n_q_heads
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    w = (torch.randn((H, cfg.d_sem, 128), generator=gen, device=dev) / cfg.d_sem ** 0.5).bfloat16()
    ov = torch.empty(out.shape[:-1] + (128,), dtype=torch.bfloat16, device=dev)
    t = time_cuda(lambda: B.latent_to_value(out, w, out=ov), 1, 3)
    nbytes = out.numel() * 2 + ov.numel() * 2 + w.numel() * 2
    fl = 2.0 * out.numel() * 128
    return dict(ms=t, bytes=nbytes, gbs=nbytes / t / 1e6, frac_of_measured_hbm=nbytes / t / 1e6 / peaks["hbm_gbs"], tflops=fl / t / 1e9)


def measure_dense_comparison(B, dev, peaks, iters=2):
    """Dense absorbed-MLA attention (Eq. 5) through the same entry point (window >= L) beside LCA on
    config 2 (the 128K dense run would take seconds per launch)."""
    cfg = I.CONFIGS["mla_32k"]
    L, g = cfg.seq_len, cfg.group_size
    inp = I.make_mla_inputs(cfg, dev)
    out = torch.empty((1, L, cfg.n_q_heads, cfg.d_sem), dtype=torch.bfloat16, device=dev)
    res = {}
    for name, w in (("lca", cfg.window), ("dense", L)):
        c2 = I.scaled(cfg, window=w)
        p = B.params_from_config(c2, batch=1)
        cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
        ws = B.workspace(p, B.LCA_WS_PREFILL, dev)
        t = time_cuda(lambda: B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"],
                                                  cond["cache_pos"], out=out, ws=ws), 2, iters)
        fl = attention_flops(c2)
        res[name] = dict(ms=t, tflops=fl / t / 1e9, flops=fl)
    res["workload"] = f"mla_32k: L={L}, H={cfg.n_q_heads}"
    res["speedup_lca_over_dense"] = res["dense"]["ms"] / res["lca"]["ms"]
    return res


def measure_scaling(B, dev, peaks, lengths=(65536, 131072, 262144, 524288, 1048576), dense_up_to=131072):
    """Context-length scaling with the paper's own hyper-parameters (g = 16, w = 1024) on a
    DeepSeek-V2-Lite-shaped layer (16 heads): prefill time of LCA and, while affordable, of dense
    absorbed MLA through the same kernel; KV-cache rows kept."""
    rows = []
    for L in lengths:
        cfg = I.scaled(I.CONFIGS["mla_32k"], name=f"v2lite_{L}", seq_len=L, group_size=16, window=1024, needle_every=4096)
        g = cfg.group_size
        inp = I.make_mla_inputs(cfg, dev)
        out = torch.empty((1, L, cfg.n_q_heads, cfg.d_sem), dtype=torch.bfloat16, device=dev)
        p = B.params_from_config(cfg, batch=1)
        m, k = B.lca_partition(p)
        cond = B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
        wsc = B.workspace(p, B.LCA_WS_CONDENSE, dev)
        t_c = time_cuda(lambda: B.condense(p, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"], out=cond, ws=wsc), 1, 2)
        t_a = time_cuda(lambda: B.prefill_attention(p, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cond["cache_sem"],
                                                    cond["cache_pos"], out=out), 1, 2)
        row = dict(seq_len=L, cache_rows=m + k, kv_reduction=1.0 - (m + k) / L, condense_ms=t_c, attention_ms=t_a,
                   attention_tflops=attention_flops(cfg) / t_a / 1e9, tokens_per_s=L / ((t_c + t_a) * 1e-3))
        if L <= dense_up_to:
            cd = I.scaled(cfg, window=L)
            pd = B.params_from_config(cd, batch=1)
            cdn = B.condense(pd, inp["q_sem"][L - g:], inp["q_pos"][L - g:], inp["ckv"], inp["kr"])
            t_d = time_cuda(lambda: B.prefill_attention(pd, inp["q_sem"], inp["q_pos"], inp["ckv"], inp["kr"], cdn["cache_sem"],
                                                        cdn["cache_pos"], out=out), 1, 1)
            row.update(dense_attention_ms=t_d, dense_tflops=attention_flops(cd) / t_d / 1e9, speedup_over_dense=t_d / (t_c + t_a))
        rows.append(row)
        del inp, out, cond
        torch.cuda.empty_cache()
    return dict(workload="V2-Lite-shaped layer, H=16, paper defaults g=16, w=1024", rows=rows)


def launcher_command(n_gpus: int, argv, port: int = 0):
    """The command that runs this script as `n_gpus` ranks of one node (one replica per GPU)."""
    if port <= 0:
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}", "--master-addr", "127.0.0.1",
            "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="mla_128k", choices=list(I.CONFIGS.keys()) + ["scaling", "value_projection"],
                    help="mla_128k is the benchmark; mla_1k / mla_32k run the same step on configs 1 / 2; mla_decode and "
                         "gqa_64k print the side measurements of configs 4 / 5 on their own (used for profiling)")
    ap.add_argument("--attn-impl", type=int, default=0, help="0 auto, 1 scalar kernel, 2 tensor-core kernel")
    ap.add_argument("--e2e-steps", type=int, default=9)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the decode / GQA / dense-comparison side measurements")
    ap.add_argument("--decode-batch", type=int, default=64)
    ap.add_argument("--seq-len", type=int, default=0, help="gqa_64k / value_projection: a shorter sequence of the same shape (small profiler captures)")
    ap.add_argument("--ref-rows", type=int, default=64, help="query rows in the oracle's bounded sample")
    ap.add_argument("--ref-heads", type=int, default=128, help="heads per sampled row in the oracle's sample (capped at the head count)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher around us: start the N replicas ourselves (one process per GPU) and hand over
        raise SystemExit(subprocess.call(launcher_command(args.gpus, sys.argv[1:])))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = I.CONFIGS.get(args.config, I.CONFIGS["mla_128k"])
    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    from paper_2604_12452_b200 import build
    build.build()
    from paper_2604_12452_b200 import binding as B
    B.lca_set_attention_impl(args.attn_impl)
    if args.config == "scaling":
        if rank == 0:
            torch.cuda.set_device(local_rank)
            res = measure_scaling(B, f"cuda:{local_rank}", measured_peaks())
            print(json.dumps(dict(metric="side_measurement", config=dict(workload=res["workload"]), n_gpus=1, data="synthetic",
                                  result=res, gpu_launches=None)))
        return
    if args.config == "value_projection":
        if rank == 0:
            torch.cuda.set_device(local_rank)
            dev = f"cuda:{local_rank}"
            cfg = I.scaled(I.CONFIGS["mla_128k"], seq_len=args.seq_len or 16384)
            lat = torch.randn((1, cfg.seq_len, cfg.n_q_heads, cfg.d_sem), device=dev).bfloat16()
            res = measure_value_projection(B, dev, cfg, lat, measured_peaks())
            print(json.dumps(dict(metric="side_measurement", config=dict(workload=f"value projection of {cfg.seq_len} tokens x {cfg.n_q_heads} heads"),
                                  n_gpus=1, data="synthetic", result=res, gpu_launches=None)))
        return
    if args.config in ("mla_decode", "gqa_64k"):
        if rank == 0:
            torch.cuda.set_device(local_rank)
            peaks = measured_peaks()
            dev = f"cuda:{local_rank}"
            res = (measure_decode_config(B, dev, args.decode_batch, peaks, args.warmup, args.steps) if args.config == "mla_decode"
                   else measure_gqa_config(B, dev, peaks, args.warmup, args.steps, args.seq_len))
            print(json.dumps(dict(metric="side_measurement", config=dict(workload=res["workload"]), n_gpus=1, steps=args.steps,
                                  warmup=args.warmup, data="synthetic", result=res, gpu_launches=None)))
        return
    run_ours(args, cfg, rank, world, local_rank)


if __name__ == "__main__":
    main()
