#!/usr/bin/env python
"""Benchmark of the decode hot path on B200: one "step" is one pass of the whole path for one
attention layer and one new token per sequence --

    seer_kcomp_append (the block that just filled)  ->  seer_gate_select (Q branch, scores,
    token-budget top-k)  ->  seer_sparse_decode (split-KV attention + LSE combine)

-- on the long-context sweep workload (batch 8, 40 query / 8 KV heads, head_dim 128,
KV length 131072, block 64, 90 % of the blocks skipped), with seer_dense_decode timed
beside it as the speed-up denominator.  Inputs are seeded and synthetic.  Prints ONE JSON
line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--sparsity S] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sparse_decode_selected_kv_GBps"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one sparse-decode launch, from an ncu capture of a
# quarter-size case (batch 2): 107.7 MB read + 4.2 MB written for 107.5 MB of algorithmic bytes.
# Reads grow with the selected tiles, writes (partials) with the number of CTAs, so a launch on
# `batch` sequences moves about batch/2 * 107.7 MB + 4.2 MB.
NCU_READ_BYTES_PER_2_SEQUENCES = 107.697e6
NCU_WRITE_BYTES_PER_LAUNCH = 4.21e6


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self._nvml
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)
        out = {"sm_mhz": int(np.median(self.samples)) if self.samples else None,
               "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        return out


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ---- the multi-GPU part: ranks are replicas with their own batches, no data-path collective ----
def init_ranks(backend: str, device=None):
    """(rank, world, local_rank) from the torchrun environment; starts the process group if world > 1."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if device is not None else {}
        dist.init_process_group(backend, **kw)
    return rank, world, local


def rank_seed(rank: int) -> int:
    """Every rank decodes its own batch of sequences."""
    from paper_2506_08889_b200 import synth
    return synth.BASE_SEED + 1000 * rank


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the job is as slow as its slowest rank)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def repeat_blocks(timed_block, n, min_s, max_repeats=200, device="cpu"):
    """Repeats `timed_block(n)` (ms per call of a block of n calls) until `min_s` seconds have been timed;
    returns (median block, number of blocks).  Every block's time is first replaced by its maximum over the
    ranks, so that all ranks see the same numbers and stop after the same block -- the blocks contain
    barriers, and ranks that went on for different numbers of blocks would wait for one another forever."""
    import numpy as np
    blocks, total = [], 0.0
    while not blocks or (total < min_s and len(blocks) < max_repeats):
        ms = max_over_ranks([timed_block(n)], device)[0]
        blocks.append(ms)
        total += ms * n * 1e-3
    return float(np.median(blocks)), len(blocks)


def job_throughput_gbs(world: int, bytes_per_rank: int, ms: float) -> float:
    """Whole-job GB/s: all ranks' bytes over the slowest rank's time."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


# --------------------------------------------------------------------------------------------
def build_layers(w, n_layers, seed, dev):
    """Per layer: K/V cache (K doubles as the pre-RoPE keys the gate pools), gate weights,
    compressed-K cache (built in bulk by the library, untimed), queries."""
    import torch
    from paper_2506_08889_b200 import binding, synth
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    layers = []
    for l in range(n_layers):
        tag = f"{w.name}:L{l}:"
        lay = {
            "k": synth.normal_bf16((B, Hkv, L, d), seed, tag + "k", dev),
            "v": synth.normal_bf16((B, Hkv, L, d), seed, tag + "v", dev),
            "q": synth.normal_bf16((B, Hq, d), seed, tag + "q", dev),
            "qn": synth.normal_bf16((B, Hq, d), seed, tag + "qn", dev),
            "wq": synth.normal_bf16((Hkv, w.d_gate, w.group * d), seed, tag + "wq", dev, std=w.gate_weight_std),
            "wk": synth.normal_bf16((Hkv, w.d_gate, 3 * d), seed, tag + "wk", dev, std=w.gate_weight_std),
            "kc": torch.zeros((B, Hkv, L // b, w.d_gate), dtype=torch.bfloat16, device=dev),
        }
        layers.append(lay)
    return layers


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2506_08889_b200 import binding, synth

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    rank, world, local = init_ranks("nccl", torch.device(dev))

    w = synth.workload(4)
    w.sparsity = args.sparsity
    if args.batch:
        w.batch = args.batch                        # smaller cases for profiler captures
    if args.seq_len:
        w.seq_len = args.seq_len
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    n_blocks = L // b
    k_sel = w.keep(n_blocks)
    budget = k_sel * b
    seed = rank_seed(rank)
    n_layers = args.layers
    layers = build_layers(w, n_layers, seed, dev)

    ctx = binding.Context(local)
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    lens_t = torch.full((B,), L, dtype=torch.int32, device=dev)
    idx = torch.zeros((B, Hkv, k_sel), dtype=torch.int32, device=dev)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=dev)
    out_dense = torch.zeros_like(out)
    for lay in layers:
        lay["gate"] = binding.make_gate(w.d_gate, w.rope_theta, lay["wq"], lay["wk"], lay["kc"], n_blocks)
        lay["kv"] = binding.make_kv(lay["k"], lay["v"], lens_t)
        # compressed keys of all blocks but the one the timed step appends
        ctx.seer_kcomp_append(shape, lay["gate"], lens_t, lay["k"], first_block=0, num_blocks=n_blocks - 1)
    torch.cuda.synchronize()

    stream = torch.cuda.current_stream()

    def step(lay, ev=None):
        if ev is None:
            # the call a user makes: one step of one layer (append: L % b == 0, so every sequence appends)
            ctx.seer_decode_step(shape, lay["kv"], lay["gate"], lay["q"], lay["qn"], lay["k"], budget,
                                 idx, cnt, k_sel, out, stream=stream)
            return
        # the same three kernels through the separate entry points, with the decode launch bracketed
        ctx.seer_kcomp_append(shape, lay["gate"], lens_t, lay["k"], stream=stream)
        ctx.seer_gate_select(shape, lay["gate"], lens_t, lay["qn"], None, budget, idx, cnt, k_sel, stream=stream)
        ev[0].record()
        ctx.seer_sparse_decode(shape, lay["kv"], lay["q"], idx, cnt, k_sel, out, stream=stream)
        ev[1].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # algorithmic bytes of one step (what the method itself must move)
    sel_kv_bytes = B * Hkv * k_sel * b * d * 2 * 2
    decode_bytes = sel_kv_bytes + 2 * B * Hq * d * 2 + 4 * B * Hkv * k_sel
    gate_bytes = B * Hkv * (n_blocks - 1) * w.d_gate * 2 + Hkv * w.d_gate * w.group * d * 2 + 2 * 4 * B * Hkv * (n_blocks - 1)
    kcomp_bytes = B * Hkv * b * d * 2 + Hkv * w.d_gate * 3 * d * 2 + B * Hkv * w.d_gate * 2
    dense_bytes = B * Hkv * L * d * 2 * 2 + 2 * B * Hq * d * 2

    K, W = args.steps, max(args.warmup, 3)
    for s in range(W):
        step(layers[s % n_layers])
        ctx.seer_dense_decode(shape, layers[s % n_layers]["kv"], layers[s % n_layers]["q"], out_dense)
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.SEER_OK

    # ---- timed region: blocks of exactly K steps, device timed, max over ranks ---------------
    # A block of K steps is timed as one region (barrier + synchronize on both sides, events on the
    # stream); the block is repeated until at least `min_timed_s` seconds have been timed and the
    # median block is reported, so that a small --steps gives the same figure as a large one.
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()

    def timed_block(fn, n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for s in range(n):
            fn(s)
        e1.record()
        barrier()
        return e0.elapsed_time(e1) / n

    def repeated(fn, n, min_s=None, max_repeats=200):
        """Median over repeated blocks of n calls (ms per call), and the number of blocks."""
        min_s = args.min_timed_s if min_s is None else min_s
        return repeat_blocks(lambda m: timed_block(fn, m), n, min_s, max_repeats, dev)

    launches0 = ctx.launch_count()
    step_ms, repeats = repeated(lambda s: step(layers[s % n_layers]), K)
    launches = (ctx.launch_count() - launches0) // repeats
    # The sparse-decode launch bracketed by events, in a pass of its own (an event record between two
    # kernels keeps the second from starting its set-up under the first one's tail, so bracketed steps
    # are kept out of the step timing): at least 32 samples, median.
    n_ev = max(32, min(K, 256))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
    barrier()
    for s in range(n_ev):
        step(layers[s % n_layers], evs[s])
    barrier()
    sparse_ms = float(np.median([a.elapsed_time(bq) for a, bq in evs]))
    # what two event records cost around a launch that does next to nothing (a one-element fill), taken the same way:
    # the part of the bracketed figure above that belongs to the bracketing, reported beside it, never subtracted
    tiny = torch.zeros(1, dtype=torch.int32, device=dev)
    barrier()
    for s in range(n_ev):
        step(layers[s % n_layers])
        evs[s][0].record()
        tiny.fill_(1)
        evs[s][1].record()
    barrier()
    empty_ms = float(np.median([a.elapsed_time(bq) for a, bq in evs]))

    # dense decode on the same tensors (speed-up denominator), same protocol
    Kd = max(8, min(K, 200))
    dense_ms, _ = repeated(lambda s: ctx.seer_dense_decode(shape, layers[s % n_layers]["kv"], layers[s % n_layers]["q"],
                                                           out_dense), Kd)
    # sparse kernel alone, back to back (no events inside), for the kernel-only speed-up
    sparse_b2b_ms, _ = repeated(lambda s: ctx.seer_sparse_decode(shape, layers[s % n_layers]["kv"], layers[s % n_layers]["q"],
                                                                 idx, cnt, k_sel, out), K)
    # the step without the compressed-K update (63 steps of 64 in a real decode: a block fills once per b tokens)
    step_noappend_ms, _ = repeated(lambda s: ctx.seer_decode_step(shape, layers[s % n_layers]["kv"], layers[s % n_layers]["gate"],
                                                                  layers[s % n_layers]["q"], layers[s % n_layers]["qn"], None,
                                                                  budget, idx, cnt, k_sel, out, stream=stream), K)
    # the bulk build of the compressed-K cache after prefill (all blocks but the last), one layer per launch
    bulk_ms, _ = repeated(lambda s: ctx.seer_kcomp_append(shape, layers[s % n_layers]["gate"], lens_t, layers[s % n_layers]["k"],
                                                          first_block=0, num_blocks=n_blocks - 1, stream=stream),
                          max(4, min(K, 8 * n_layers)))
    # what a kernel that only reads gets out of this GPU's memory: the library's read probe over one layer's K and V
    # caches per launch (4.3 GB, rotating over the layers), the ceiling the decode kernels' figures are set against
    probe_chk = torch.zeros(1, dtype=torch.int64, device=dev)
    probe_bytes = layers[0]["k"].numel() * 2

    def probe(s):
        lay = layers[s % n_layers]
        ctx.seer_debug_read_bandwidth(lay["k"], probe_bytes, probe_chk, stream=stream)
        ctx.seer_debug_read_bandwidth(lay["v"], probe_bytes, probe_chk, stream=stream)

    probe_ms, _ = repeated(probe, max(4, min(K, 4 * n_layers)))
    probe_gbs = 2 * probe_bytes / (probe_ms * 1e-3) / 1e9
    clocks = sampler.stop()

    # ---- end to end through the same API with host buffers ----------------------------------
    # Per-step inputs (queries, pre-RoPE queries, the new token's K and V rows, lengths) start in
    # pinned host memory; the result is read back to the host.  The KV cache is device state.
    # one pinned staging buffer and one device buffer hold all per-step inputs, so a step is one H2D copy
    parts = [("q", layers[0]["q"]), ("qn", layers[0]["qn"]),
             ("k_new", layers[0]["k"][:, :, L - 1, :].contiguous()), ("v_new", layers[0]["v"][:, :, L - 1, :].contiguous()),
             ("lens", lens_t)]
    offs, total = {}, 0
    for name, t in parts:
        offs[name] = total
        total += (t.numel() * t.element_size() + 255) // 256 * 256
    hbuf = torch.empty(total, dtype=torch.uint8).pin_memory()
    dbuf = torch.empty(total, dtype=torch.uint8, device=dev)

    def view(buf, name, like):
        n = like.numel() * like.element_size()
        return buf[offs[name]:offs[name] + n].view(like.dtype).view(like.shape)

    for name, t in parts:
        view(hbuf, name, t).copy_(t)
    dq, dqn = view(dbuf, "q", parts[0][1]), view(dbuf, "qn", parts[1][1])
    dk_new, dv_new = view(dbuf, "k_new", parts[2][1]), view(dbuf, "v_new", parts[3][1])
    dlens = view(dbuf, "lens", lens_t)
    hout = torch.empty((B, Hq, d), dtype=torch.bfloat16).pin_memory()
    h2d = sum(t.numel() * t.element_size() for _, t in parts)
    d2h = hout.numel() * hout.element_size()

    def e2e_step(lay):
        dbuf.copy_(hbuf, non_blocking=True)          # q, q_nope, the new token's K and V rows, lengths
        lay["k_last"].copy_(dk_new)                  # the caller's append of the new token
        lay["v_last"].copy_(dv_new)
        ctx.seer_decode_step(shape, lay["kv_e2e"], lay["gate"], dq, dqn, lay["k"], budget, idx, cnt, k_sel, out,
                             stream=stream)
        hout.copy_(out, non_blocking=True)
        stream.synchronize()

    for lay in layers:
        lay["kv_e2e"] = binding.make_kv(lay["k"], lay["v"], dlens)
        lay["k_last"], lay["v_last"] = lay["k"][:, :, L - 1, :], lay["v"][:, :, L - 1, :]   # (views: the rows the step appends)
    Ke = max(8, min(K, 300))
    for s in range(3):
        e2e_step(layers[s % n_layers])
    def e2e_block(n):
        barrier()
        w0 = time.perf_counter()
        for s in range(n):
            e2e_step(layers[s % n_layers])
        barrier()
        return (time.perf_counter() - w0) * 1e3 / n

    e2e_ms, _ = repeat_blocks(e2e_block, Ke, args.min_timed_s, 200, dev)
    assert ctx.device_status() == binding.SEER_OK

    # ---- reduce over ranks -------------------------------------------------------------------
    step_ms, sparse_ms, dense_ms, sparse_b2b_ms, e2e_ms, step_noappend_ms, bulk_ms = max_over_ranks(
        [step_ms, sparse_ms, dense_ms, sparse_b2b_ms, e2e_ms, step_noappend_ms, bulk_ms], dev)

    result = None
    if rank == 0:
        peak, peak_kind = measured_hbm_peak()
        value = job_throughput_gbs(world, sel_kv_bytes, step_ms)
        kern_gbs = decode_bytes / (sparse_ms * 1e-3) / 1e9
        result = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "repeats": repeats,
            "ms_per_step": round(step_ms, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "batch_per_gpu": B, "num_q_heads": Hq, "num_kv_heads": Hkv,
                       "head_dim": d, "seq_len": L, "block_size": b, "sparsity": args.sparsity,
                       "selected_blocks": k_sel, "of_blocks": n_blocks, "parallelism": f"replicated-batches x{world}",
                       "step": "seer_decode_step = kcomp_append + gate_select + sparse_decode (one layer, one token per sequence)",
                       "l2": f"steps rotate over {n_layers} layer caches ({n_layers * dense_bytes / 1e9:.1f} GB), "
                             f"selected bytes per step {sel_kv_bytes / 1e6:.0f} MB > L2"},
            "e2e": {"value": round(job_throughput_gbs(world, sel_kv_bytes, e2e_ms), 1), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 5)},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "decode_kernel<sparse>", "achieved": round(kern_gbs, 1),
                         "peak": peak, "unit": "GB/s", "frac": round(kern_gbs / peak, 4), "peak_kind": f"of {peak_kind}",
                         "frac_of_nominal_8000": round(kern_gbs / NOMINAL_HBM_GBS, 4),
                         "algorithmic_bytes_per_launch": decode_bytes, "us_per_launch": round(sparse_ms * 1e3, 2),
                         "event_samples": n_ev, "empty_launch_between_events_us": round(empty_ms * 1e3, 2),
                         "traffic": (int(NCU_READ_BYTES_PER_2_SEQUENCES * B / 2 * (1.0 - args.sparsity) / 0.1
                                         + NCU_WRITE_BYTES_PER_LAUNCH) if abs(args.sparsity - 0.9) < 1e-9 else None),
                         "traffic_note": "ncu capture at batch 2, scaled by the units processed",
                         # the same kernel launched back to back (no event between launches, so that each
                         # launch's set-up overlaps its predecessor's tail as it does inside the step)
                         "us_per_launch_back_to_back": round(sparse_b2b_ms * 1e3, 2),
                         "frac_back_to_back": round(decode_bytes / (sparse_b2b_ms * 1e-3) / 1e9 / peak, 4),
                         # against what a read-only kernel reaches on this GPU (the library's probe, same run)
                         "read_probe_GBps": round(probe_gbs, 1),
                         "frac_of_read_probe": round(kern_gbs / probe_gbs, 4),
                         "frac_back_to_back_of_read_probe": round(decode_bytes / (sparse_b2b_ms * 1e-3) / 1e9 / probe_gbs, 4)},
            "extra": {
                "tokens_per_s_per_layer": round(world * B / (step_ms * 1e-3), 1),
                "selected_kv_bytes_per_step": sel_kv_bytes,
                "step_algorithmic_bytes": decode_bytes + gate_bytes + kcomp_bytes,
                "sparse_kernel_us": round(sparse_ms * 1e3, 2), "sparse_kernel_back_to_back_us": round(sparse_b2b_ms * 1e3, 2),
                "dense_kernel_us": round(dense_ms * 1e3, 2),
                "dense_kernel_GBps": round(dense_bytes / (dense_ms * 1e-3) / 1e9, 1),
                "dense_frac_of_measured_peak": round(dense_bytes / (dense_ms * 1e-3) / 1e9 / peak, 4),
                "gate_plus_kcomp_us": round((step_ms - sparse_ms) * 1e3, 2),
                "step_without_append_us": round(step_noappend_ms * 1e3, 2),
                "speedup_vs_dense_kernel": round(dense_ms / sparse_b2b_ms, 3),
                "speedup_vs_dense_step": round(dense_ms / step_ms, 3),
                "ideal_speedup": round(n_blocks / k_sel, 3),
                # bulk build of the compressed-K cache: the keys read once (the algorithmic bytes) over the launch time
                "bulk_kcomp_us": round(bulk_ms * 1e3, 1),
                "bulk_kcomp_GBps": round(B * Hkv * (n_blocks - 1) * b * d * 2 / (bulk_ms * 1e-3) / 1e9, 1),
                "bulk_kcomp_frac_of_measured_peak": round(B * Hkv * (n_blocks - 1) * b * d * 2 / (bulk_ms * 1e-3) / 1e9 / peak, 4),
            },
        }
        if not args.no_cpu_baseline and world == 1:
            result["cpu_baseline"] = cpu_baseline(w, layers[0], k_sel, budget, sel_kv_bytes, seconds=args.cpu_seconds)
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(result))


# --------------------------------------------------------------------------------------------
def run_sweep(args):
    """Sparsity sweep of the long-context workload (kernel-only times, one GPU): sparse decode at
    each sparsity level against the dense kernel on the same tensors.  Writes one JSON document."""
    import torch
    from paper_2506_08889_b200 import binding, synth
    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = synth.workload(4)
    if args.batch:
        w.batch = args.batch
    if args.seq_len:
        w.seq_len = args.seq_len
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    n_blocks = L // b
    n_layers = args.layers
    layers = build_layers(w, n_layers, synth.BASE_SEED, dev)
    ctx = binding.Context(0)
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    lens_t = torch.full((B,), L, dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=dev)
    for lay in layers:
        lay["kv"] = binding.make_kv(lay["k"], lay["v"], lens_t)
    peak, peak_kind = measured_hbm_peak()
    K = args.steps

    def timed(fn, iters):
        for s in range(5):
            fn(s)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in range(iters):
            fn(s)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3      # us

    dense_us = timed(lambda s: ctx.seer_dense_decode(shape, layers[s % n_layers]["kv"], layers[s % n_layers]["q"], out),
                     max(8, K // 10))
    dense_bytes = B * Hkv * L * d * 4
    rows = []
    for sp in (0.0, 0.5, 0.75, 0.9, 0.95):
        k_sel = synth.keep_count(n_blocks, sp)
        scores = synth.normal_f32((B, Hkv, n_blocks), synth.BASE_SEED, f"sweep:{sp}", dev)
        idx = torch.zeros((B, Hkv, k_sel), dtype=torch.int32, device=dev)
        cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
        gate = binding.make_gate(w.d_gate, w.rope_theta, None, None, None, n_blocks)
        ctx.seer_gate_select(shape, gate, lens_t, None, scores, k_sel * b, idx, cnt, k_sel)
        us = timed(lambda s: ctx.seer_sparse_decode(shape, layers[s % n_layers]["kv"], layers[s % n_layers]["q"],
                                                    idx, cnt, k_sel, out), K)
        sel_bytes = B * Hkv * k_sel * b * d * 4
        rows.append({"sparsity": sp, "selected_blocks": k_sel, "of_blocks": n_blocks, "sparse_us": round(us, 2),
                     "selected_kv_MB": round(sel_bytes / 1e6, 1), "GBps": round(sel_bytes / us / 1e3, 1),
                     "frac_of_measured_peak": round(sel_bytes / us / 1e3 / peak, 4),
                     "frac_of_8000": round(sel_bytes / us / 1e3 / NOMINAL_HBM_GBS, 4),
                     "speedup_vs_dense": round(dense_us / us, 3), "ideal_speedup": round(n_blocks / k_sel, 3)})
    assert ctx.device_status() == binding.SEER_OK
    doc = {"workload": w.name, "batch": B, "seq_len": L, "layers_rotated": n_layers, "dense_us": round(dense_us, 2),
           "dense_GBps": round(dense_bytes / dense_us / 1e3, 1), "peak_GBps": peak, "peak_kind": peak_kind, "rows": rows}
    print(json.dumps(doc))
    ctx.close()


def run_multi(args):
    """Multi-query-token decode (q_len tokens per sequence over one block list) on the long-context
    workload's cache at the given sparsity, kernel-only, one GPU: time per call and per token for
    q_len = 1..8 and three group sizes.  Writes one JSON document."""
    import torch
    from paper_2506_08889_b200 import binding, synth
    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = synth.workload(4)
    w.sparsity = args.sparsity
    if args.batch:
        w.batch = args.batch
    if args.seq_len:
        w.seq_len = args.seq_len
    B, Hkv, d, b, L = w.batch, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    n_blocks = L // b
    k_sel = w.keep(n_blocks)
    n_layers = args.layers
    layers = build_layers(w, n_layers, synth.BASE_SEED, dev)
    ctx = binding.Context(0)
    lens_t = torch.full((B,), L, dtype=torch.int32, device=dev)
    lens = np.full(B, L, np.int32)
    for l, lay in enumerate(layers):
        lay["kv"] = binding.make_kv(lay["k"], lay["v"], lens_t)
        idx, cnt = synth.random_block_lists(lens, Hkv, b, k_sel, k_sel, synth.BASE_SEED, f"multi:{l}")
        lay["idx"], lay["cnt"] = torch.as_tensor(idx, device=dev), torch.as_tensor(cnt, device=dev)
    sel_bytes = B * Hkv * k_sel * b * d * 4
    rows = []
    for Hq in (32, 40, 64):
        shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
        for T in (1, 2, 3, 4, 8):
            q = synth.normal_bf16((B, T, Hq, d), synth.BASE_SEED, f"multi:q:{Hq}:{T}", dev)
            out = torch.zeros_like(q)

            def step(s):
                lay = layers[s % n_layers]
                ctx.seer_sparse_decode_multi(shape, lay["kv"], q, T, lay["idx"], lay["cnt"], k_sel, out)
            for s in range(5):
                step(s)
            torch.cuda.synchronize()
            n0 = ctx.launch_count()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for s in range(args.steps):
                step(s)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) / args.steps * 1e3
            launches = (ctx.launch_count() - n0) // args.steps
            rows.append({"num_q_heads": Hq, "q_len": T, "rows_per_unit": T * Hq // Hkv, "launches": launches,
                         "us_per_call": round(us, 2), "us_per_token": round(us / T, 2),
                         "GBps_read": round(launches * sel_bytes / us / 1e3, 1)})
    assert ctx.device_status() == binding.SEER_OK
    print(json.dumps({"workload": w.name, "batch": B, "seq_len": L, "sparsity": args.sparsity, "selected_blocks": k_sel,
                      "selected_kv_MB_per_launch": round(sel_bytes / 1e6, 1), "rows": rows}))
    ctx.close()


def run_grid(args):
    """The paper's own kernel-benchmark shape (Sec. 4.4): 64 query / 8 KV heads, head_dim 128, over
    sequence length x batch x sparsity, sparse kernel against the dense kernel on the same tensors.
    Kernel-only, one GPU, one JSON document; L2 is kept cold by rotating over distinct caches."""
    import torch
    from paper_2506_08889_b200 import binding, synth
    dev = "cuda:0"
    torch.cuda.set_device(0)
    ctx = binding.Context(0)
    peak, peak_kind = measured_hbm_peak()
    Hq, Hkv, d, b = 64, 8, 128, args.block_size
    rows = []

    def timed(fn, iters):
        for s in range(3):
            fn(s)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in range(iters):
            fn(s)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3

    for L in (8192, 32768, 131072):
        for B in (1, 4, 16):
            kv_bytes = B * Hkv * L * d * 4
            n_copies = max(2, min(8, int(2 * 256e6 // kv_bytes) + 1))     # rotate over > 2x L2
            caches = []
            for c in range(n_copies):
                tag = f"grid:{L}:{B}:{c}:"
                k = synth.normal_bf16((B, Hkv, L, d), synth.BASE_SEED, tag + "k", dev)
                v = synth.normal_bf16((B, Hkv, L, d), synth.BASE_SEED, tag + "v", dev)
                caches.append((k, v))
            q = synth.normal_bf16((B, Hq, d), synth.BASE_SEED, f"grid:{L}:{B}:q", dev)
            out = torch.zeros_like(q)
            lens_t = torch.full((B,), L, dtype=torch.int32, device=dev)
            shape = binding.make_shape(B, Hq, Hkv, d, b, 1.0 / float(np.sqrt(d)))
            kvs = [binding.make_kv(k, v, lens_t) for k, v in caches]
            iters = max(20, min(args.steps, int(3e5 / max(1.0, kv_bytes / 6e6))))
            dense_us = timed(lambda s: ctx.seer_dense_decode(shape, kvs[s % n_copies], q, out), max(5, iters // 4))
            nb = L // b
            for sp in (0.5, 0.7, 0.9):
                k_sel = synth.keep_count(nb, sp)
                scores = synth.normal_f32((B, Hkv, nb), synth.BASE_SEED, f"grid:{L}:{B}:{sp}", dev)
                idx = torch.zeros((B, Hkv, k_sel), dtype=torch.int32, device=dev)
                cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
                gate = binding.make_gate(128, 1.0e6, None, None, None, nb)
                ctx.seer_gate_select(shape, gate, lens_t, None, scores, k_sel * b, idx, cnt, k_sel)
                us = timed(lambda s: ctx.seer_sparse_decode(shape, kvs[s % n_copies], q, idx, cnt, k_sel, out), iters)
                sel = B * Hkv * k_sel * b * d * 4
                rows.append({"seq_len": L, "batch": B, "sparsity": sp, "sparse_us": round(us, 2),
                             "dense_us": round(dense_us, 2), "speedup": round(dense_us / us, 2),
                             "ideal": round(nb / k_sel, 2), "GBps": round(sel / us / 1e3, 1)})
            del caches, kvs
            torch.cuda.empty_cache()
    assert ctx.device_status() == binding.SEER_OK
    print(json.dumps({"shape": "64 query / 8 KV heads, head_dim 128", "block_size": b, "peak_GBps": peak,
                      "peak_kind": peak_kind, "rows": rows}))
    ctx.close()


def run_workloads(args):
    """The other specified workloads, one GPU, one JSON document: the batch-1 8B and 14B shapes (a
    launch moves 16 MiB, less than L2 holds and about as long as a launch takes) each timed (i) alone --
    one call, L2 flushed before it, event-bracketed -- and (ii) as a stream over `layers` distinct
    layer caches (more than twice L2 in total), which is the figure compared with the HBM roofline;
    and the ragged batch of 16 at block size 128.  Beside each: the library's own dense kernel under
    the same protocol, and the fp64 oracle's time for the same call on the host cores."""
    import torch
    import oracle
    from paper_2506_08889_b200 import binding, synth
    dev = "cuda:0"
    torch.cuda.set_device(0)
    ctx = binding.Context(0)
    peak, peak_kind = measured_hbm_peak()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)        # > 2 x L2
    rows = []

    def isolated(fn, n=40):
        """Median of single calls, each after an L2 flush, bracketed by events (us)."""
        fn(0)
        ts = []
        for s in range(n):
            flush.fill_(s & 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(s)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) * 1e3)
        return float(np.median(ts))

    def streamed(fn, n):
        """Calls back to back over the distinct layers (us per call, median of repeated blocks)."""
        for s in range(n):
            fn(s)
        blocks, total = [], 0.0
        while not blocks or (total < args.min_timed_s and len(blocks) < 100):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for s in range(n):
                fn(s)
            e1.record()
            torch.cuda.synchronize()
            blocks.append(e0.elapsed_time(e1) / n * 1e3)
            total += blocks[-1] * n * 1e-6
        return float(np.median(blocks))

    def row(w, what, sel_bytes, us_iso, us_stream, dense_bytes, dense_iso, dense_stream, extra):
        r = {"workload": w.name, "call": what, "selected_kv_MB": round(sel_bytes / 1e6, 2),
             "isolated_us": round(us_iso, 2), "streamed_us": round(us_stream, 2),
             "streamed_GBps": round(sel_bytes / us_stream / 1e3, 1),
             "streamed_frac_of_measured_peak": round(sel_bytes / us_stream / 1e3 / peak, 4),
             "streamed_frac_of_8000": round(sel_bytes / us_stream / 1e3 / NOMINAL_HBM_GBS, 4),
             "isolated_GBps": round(sel_bytes / us_iso / 1e3, 1),
             "dense_isolated_us": round(dense_iso, 2), "dense_streamed_us": round(dense_stream, 2),
             "dense_streamed_GBps": round(dense_bytes / dense_stream / 1e3, 1),
             "speedup_vs_dense_streamed": round(dense_stream / us_stream, 3),
             "speedup_vs_dense_isolated": round(dense_iso / us_iso, 3)}
        r.update(extra)
        rows.append(r)

    # ---- batch 1, Qwen3-8B shape: selection on given scores, then sparse decode ---------------------
    w = synth.workload(1)
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    nb, k_sel, NL = L // b, w.keep(L // b), args.stream_layers
    lens_t = torch.full((B,), L, dtype=torch.int32, device=dev)
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    lay = []
    for l in range(NL):
        tag = f"{w.name}:L{l}:"
        k = synth.normal_bf16((B, Hkv, L, d), synth.BASE_SEED, tag + "k", dev)
        v = synth.normal_bf16((B, Hkv, L, d), synth.BASE_SEED, tag + "v", dev)
        lay.append({"kv": binding.make_kv(k, v, lens_t), "k": k, "v": v,
                    "q": synth.normal_bf16((B, Hq, d), synth.BASE_SEED, tag + "q", dev),
                    "sc": synth.normal_f32((B, Hkv, nb), synth.BASE_SEED, tag + "scores", dev)})
    gate0 = binding.make_gate(w.d_gate, w.rope_theta, None, None, None, nb)
    idx = torch.zeros((B, Hkv, k_sel), dtype=torch.int32, device=dev)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=dev)
    ctx.seer_gate_select(shape, gate0, lens_t, None, lay[0]["sc"], w.token_budget, idx, cnt, k_sel)

    def dec(s):
        ctx.seer_sparse_decode(shape, lay[s % NL]["kv"], lay[s % NL]["q"], idx, cnt, k_sel, out)

    def sel_dec(s):
        ctx.seer_gate_select(shape, gate0, lens_t, None, lay[s % NL]["sc"], w.token_budget, idx, cnt, k_sel)
        ctx.seer_sparse_decode(shape, lay[s % NL]["kv"], lay[s % NL]["q"], idx, cnt, k_sel, out)

    def dense(s):
        ctx.seer_dense_decode(shape, lay[s % NL]["kv"], lay[s % NL]["q"], out)

    sel_bytes = B * Hkv * k_sel * b * d * 4
    dense_bytes = B * Hkv * L * d * 4
    d_iso, d_str = isolated(dense), streamed(dense, NL)
    # the oracle on the same call: all host threads, and one thread
    hk, hv, hq = synth.bf16_bits(lay[0]["k"]), synth.bf16_bits(lay[0]["v"]), synth.bf16_bits(lay[0]["q"])
    hsc = lay[0]["sc"].cpu().numpy()
    lens = np.full(B, L, np.int32)

    def oracle_call():
        i2, c2 = oracle.select(hsc, lens, b, w.token_budget, k_sel)
        oracle.sparse(hq, hk, hv, lens, i2, c2, b, w.sm_scale)
    oracle_call()
    t0 = time.perf_counter(); oracle_call(); o_all = time.perf_counter() - t0
    n_thr = oracle.num_threads()
    oracle.set_num_threads(1)
    t0 = time.perf_counter(); oracle_call(); o_one = time.perf_counter() - t0
    oracle.set_num_threads(n_thr)
    row(w, "seer_sparse_decode", sel_bytes, isolated(dec), streamed(dec, NL), dense_bytes, d_iso, d_str,
        {"layers_streamed": NL, "oracle_ms_all_threads": round(o_all * 1e3, 2), "oracle_threads": n_thr,
         "oracle_ms_one_thread": round(o_one * 1e3, 2)})
    row(w, "seer_gate_select(scores) + seer_sparse_decode", sel_bytes, isolated(sel_dec), streamed(sel_dec, NL),
        dense_bytes, d_iso, d_str, {"layers_streamed": NL})
    del lay
    torch.cuda.empty_cache()

    # ---- batch 1, Qwen3-14B shape: the whole step (append + gate + sparse decode) ---------------------
    w = synth.workload(2)
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    nb, k_sel = L // b, w.keep(L // b)
    budget = k_sel * b
    lens_t = torch.full((B,), L, dtype=torch.int32, device=dev)
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    layers = build_layers(w, NL, synth.BASE_SEED, dev)
    idx = torch.zeros((B, Hkv, k_sel), dtype=torch.int32, device=dev)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=dev)
    for la in layers:
        la["gate"] = binding.make_gate(w.d_gate, w.rope_theta, la["wq"], la["wk"], la["kc"], nb)
        la["kv"] = binding.make_kv(la["k"], la["v"], lens_t)
        ctx.seer_kcomp_append(shape, la["gate"], lens_t, la["k"], first_block=0, num_blocks=nb - 1)
    torch.cuda.synchronize()

    def step(s):
        la = layers[s % NL]
        ctx.seer_decode_step(shape, la["kv"], la["gate"], la["q"], la["qn"], la["k"], budget, idx, cnt, k_sel, out)

    def step_noappend(s):
        la = layers[s % NL]
        ctx.seer_decode_step(shape, la["kv"], la["gate"], la["q"], la["qn"], None, budget, idx, cnt, k_sel, out)

    def dec3(s):
        la = layers[s % NL]
        ctx.seer_sparse_decode(shape, la["kv"], la["q"], idx, cnt, k_sel, out)

    def dense3(s):
        la = layers[s % NL]
        ctx.seer_dense_decode(shape, la["kv"], la["q"], out)

    step(0)
    sel_bytes = B * Hkv * k_sel * b * d * 4
    dense_bytes = B * Hkv * L * d * 4
    gate_bytes = B * Hkv * (nb - 1) * w.d_gate * 2 + Hkv * w.d_gate * w.group * d * 2
    d_iso, d_str = isolated(dense3), streamed(dense3, NL)
    host = host_copy(layers[0])
    host["kc"], _ = oracle.kcomp(host["k"], host["wk"], b, 0, nb - 1, nb, w.rope_theta)
    oracle_step(w, host, 1, Hkv, budget, k_sel)
    t0 = time.perf_counter(); oracle_step(w, host, 1, Hkv, budget, k_sel); o_all = time.perf_counter() - t0
    row(w, "seer_decode_step (append + gate + sparse decode)", sel_bytes, isolated(step), streamed(step, NL),
        dense_bytes, d_iso, d_str, {"layers_streamed": NL, "gate_bytes_MB": round(gate_bytes / 1e6, 2),
                                    "oracle_ms_all_threads": round(o_all * 1e3, 2), "oracle_threads": oracle.num_threads()})
    row(w, "seer_decode_step without the append", sel_bytes, isolated(step_noappend), streamed(step_noappend, NL),
        dense_bytes, d_iso, d_str, {"layers_streamed": NL})
    row(w, "seer_sparse_decode", sel_bytes, isolated(dec3), streamed(dec3, NL), dense_bytes, d_iso, d_str,
        {"layers_streamed": NL})
    del layers, host
    torch.cuda.empty_cache()

    # ---- batch 16, ragged lengths, block size 128, 90 % of each sequence's blocks skipped ---------------
    w = synth.workload(3)
    B, Hq, Hkv, d, b, L = w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.block_size, w.seq_len
    lens = w.lengths()
    n_i = [-(-int(x) // b) for x in lens]
    keep = [w.keep(n) for n in n_i]
    max_sel = max(keep)
    NL4 = 3
    lens_t = torch.as_tensor(lens, device=dev)
    shape = binding.make_shape(B, Hq, Hkv, d, b, w.sm_scale)
    shape1 = binding.make_shape(1, Hq, Hkv, d, b, w.sm_scale)
    lay = []
    for l in range(NL4):
        tag = f"{w.name}:L{l}:"
        k = synth.normal_bf16((B, Hkv, L, d), synth.BASE_SEED, tag + "k", dev)
        v = synth.normal_bf16((B, Hkv, L, d), synth.BASE_SEED, tag + "v", dev)
        lay.append({"kv": binding.make_kv(k, v, lens_t, max_seq_len=L), "k": k, "v": v,
                    "q": synth.normal_bf16((B, Hq, d), synth.BASE_SEED, tag + "q", dev)})
    scores = synth.normal_f32((B, Hkv, L // b), synth.BASE_SEED, w.name + ":scores", dev)
    gate4 = binding.make_gate(w.d_gate, w.rope_theta, None, None, None, L // b)
    idx = torch.full((B, Hkv, max_sel), -1, dtype=torch.int32, device=dev)
    cnt = torch.zeros((B, Hkv), dtype=torch.int32, device=dev)
    for i in range(B):                    # the kept count differs between sequences: one selection call each
        ctx.seer_gate_select(shape1, gate4, lens_t[i:i + 1], None, scores[i:i + 1], keep[i] * b, idx[i:i + 1],
                             cnt[i:i + 1], max_sel)
    torch.cuda.synchronize()
    out = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=dev)

    def dec4(s):
        ctx.seer_sparse_decode(shape, lay[s % NL4]["kv"], lay[s % NL4]["q"], idx, cnt, max_sel, out)

    def dense4(s):
        ctx.seer_dense_decode(shape, lay[s % NL4]["kv"], lay[s % NL4]["q"], out)

    sel_tokens = sum(min(int(lens[i]) - (n_i[i] - 1) * b, b) + (keep[i] - 1) * b for i in range(B))   # (an upper figure:
    # the forced last block may be partial; the other selected blocks are complete)
    sel_bytes = Hkv * sel_tokens * d * 4
    dense_bytes = Hkv * int(np.sum(lens)) * d * 4
    hq = synth.bf16_bits(lay[0]["q"])
    hk, hv = synth.bf16_bits(lay[0]["k"][:2]), synth.bf16_bits(lay[0]["v"][:2])
    i2, c2 = idx[:2].cpu().numpy(), cnt[:2].cpu().numpy()
    oracle.sparse(hq[:2], hk, hv, lens[:2], i2, c2, b, w.sm_scale)
    t0 = time.perf_counter(); oracle.sparse(hq[:2], hk, hv, lens[:2], i2, c2, b, w.sm_scale); o2 = time.perf_counter() - t0
    row(w, "seer_sparse_decode", sel_bytes, isolated(dec4, 20), streamed(dec4, 2 * NL4), dense_bytes,
        isolated(dense4, 10), streamed(dense4, NL4),
        {"layers_streamed": NL4, "lengths": [int(x) for x in lens], "selected_blocks": keep,
         "oracle_ms_all_threads_2_of_16_sequences": round(o2 * 1e3, 2), "oracle_threads": oracle.num_threads()})
    assert ctx.device_status() == binding.SEER_OK
    ctx.close()
    print(json.dumps({"peak_GBps": peak, "peak_kind": peak_kind, "rows": rows}))


def oracle_step(w, host, n_seq, n_kv_heads, budget, k_sel):
    """The whole step on the CPU oracle for the first n_seq sequences and the first
    n_kv_heads KV heads (with their query-head groups).  Returns the selected-KV bytes."""
    import oracle
    b, L, g = w.block_size, w.seq_len, w.group
    n_blocks = L // b
    lens = np.full(n_seq, L, np.int32)
    k, v = host["k"][:n_seq, :n_kv_heads], host["v"][:n_seq, :n_kv_heads]          # views
    kc = host["kc"][:n_seq, :n_kv_heads]
    wk, wq = host["wk"][:n_kv_heads], host["wq"][:n_kv_heads]
    q, qn = host["q"][:n_seq, :n_kv_heads * g], host["qn"][:n_seq, :n_kv_heads * g]
    kc, _ = oracle.kcomp(k, wk, b, n_blocks - 1, 1, n_blocks, w.rope_theta, kc_bf16=kc)
    sc, _ = oracle.scores(qn, wq, kc, [n_blocks - 1] * n_seq, [L - 1] * n_seq, w.rope_theta)
    idx, cnt = oracle.select(sc.astype(np.float32), lens, b, budget, k_sel)
    oracle.sparse(q, k, v, lens, idx, cnt, b, w.sm_scale)
    return n_seq * n_kv_heads * k_sel * b * w.head_dim * 2 * 2


def host_copy(lay):
    from paper_2506_08889_b200 import synth
    return {name: synth.bf16_bits(lay[name]) for name in ("k", "v", "q", "qn", "wq", "wk", "kc")}


def cpu_baseline(w, lay, k_sel, budget, sel_kv_bytes, seconds=15.0):
    import oracle
    host = host_copy(lay)
    H = w.num_kv_heads
    t0 = time.perf_counter()
    nbytes = oracle_step(w, host, 1, H, budget, k_sel)
    one = time.perf_counter() - t0
    n_seq = int(max(1, min(w.batch, seconds / max(one, 1e-3))))
    reps = int(max(1, min(100, seconds / max(one * n_seq, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        nbytes = oracle_step(w, host, n_seq, H, budget, k_sel)
    one = (time.perf_counter() - t0) / reps
    return {"value": round(nbytes / one / 1e9, 4), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"the whole step (kcomp + scores + select + sparse attention) for {n_seq} of {w.batch} "
                      f"sequences, all heads, {reps} repetition(s), {one:.2f} s each",
            "host_cores": os.cpu_count()}


def run_reference(args):
    """The reference arm: the fp64 oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2506_08889_b200 import synth
    w = synth.workload(4)
    w.sparsity = args.sparsity
    b, L = w.block_size, w.seq_len
    n_blocks = L // b
    k_sel = w.keep(n_blocks)
    budget = k_sel * b
    K, W = args.steps, args.warmup
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    w_small = synth.workload(4)
    w_small.batch = 1
    lay = build_layers(w_small, 1, synth.BASE_SEED, dev)[0]
    host = host_copy(lay)
    del lay
    # the compressed keys of the earlier blocks come from the oracle itself (untimed set-up)
    host["kc"], _ = oracle.kcomp(host["k"], host["wk"], b, 0, n_blocks - 1, n_blocks, w.rope_theta)
    # bounded sample: as many KV heads of one sequence per step as keep the whole run within minutes
    budget_s = 150.0
    heads = w.num_kv_heads
    while True:
        t0 = time.perf_counter()
        oracle_step(w, host, 1, heads, budget, k_sel)
        probe = time.perf_counter() - t0
        if probe * (K + W) <= budget_s or heads == 1:
            break
        heads //= 2
    K_eff = K if probe * (K + W) <= budget_s else max(1, int(budget_s / probe) - W)
    for _ in range(W):
        oracle_step(w, host, 1, heads, budget, k_sel)
    t0 = time.perf_counter()
    for _ in range(K_eff):
        nbytes = oracle_step(w, host, 1, heads, budget, k_sel)
    ms = (time.perf_counter() - t0) * 1e3 / K_eff
    value = round(nbytes / (ms * 1e-3) / 1e9, 4)
    sample = (f"one step = the whole path for 1 of {w.batch} sequences, {heads} of {w.num_kv_heads} KV heads "
              f"({heads * w.group} query heads), {K_eff} timed steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K_eff, "warmup": W, "ms_per_step": round(ms, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sparsity": args.sparsity, "selected_blocks": k_sel, "of_blocks": n_blocks,
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--sparsity", type=float, default=0.9)
    ap.add_argument("--layers", type=int, default=4, help="distinct layer caches the steps rotate over")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling cases)")
    ap.add_argument("--seq-len", type=int, default=0, help="override the workload's KV length (multiple of 64)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sweep", action="store_true", help="kernel-only sparsity sweep instead of the step benchmark")
    ap.add_argument("--grid", action="store_true", help="the paper's 64/8-head kernel grid (seq len x batch x sparsity)")
    ap.add_argument("--multi", action="store_true", help="multi-query-token decode: q_len 1..8, kernel-only")
    ap.add_argument("--block-size", type=int, default=64, help="block size for --grid (16, 32, 64 or 128)")
    ap.add_argument("--min-timed-s", type=float, default=0.2,
                    help="the block of --steps steps is repeated until this many seconds have been timed (median block reported)")
    ap.add_argument("--workloads", action="store_true",
                    help="the other specified workloads (batch-1 8B and 14B shapes, ragged batch 16): isolated and streamed")
    ap.add_argument("--stream-layers", type=int, default=32, help="distinct layer caches of the batch-1 streams (--workloads)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    args = ap.parse_args()
    if args.workloads:
        run_workloads(args)
    elif args.grid:
        run_grid(args)
    elif args.multi:
        run_multi(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
