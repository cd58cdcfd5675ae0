#!/usr/bin/env python
"""Benchmark of the hybrid-attention hot path at the 832x480 latent shape.

A step = one 3-frame chunk through the full-depth attention stack: for each of 30 layers, 4 denoising-step
forwards (pool + select + sparse SWA + history read-out + merge) and one cache commit (evict -> state absorb
-> append).  Metric: attention-only latent frames/s.  Inputs are seeded synthetic bf16 N(0,1) tensors.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun): every rank runs an independent replica (the path has no exchange step); the timed
region is bracketed by barriers, the time is the max over ranks, the value the sum of frames over ranks.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_10103_b200 import inputs as gen, replicas  # noqa: E402

METRIC = "hybrid-attn latent frames/s at 832x480 shape"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the attention kernel (history term inside) at this
# workload's layer shape, from an ncu capture of that kernel; None when the kernel has changed since the capture.
SWA_DRAM_BYTES_PER_LAUNCH = 107.3e6
UNIT = "latent frames/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.t.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i] == "Active" for r in self.rows)]
        pw = [float(r[2]) for r in self.rows if len(r) >= 7 and r[2].replace(".", "").isdigit()]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": reasons}


# ----------------------------------------------------------------------------------------------- oracle arm
ORACLE_QBLOCKS = 3        # query blocks per sampled forward: first, middle, the ragged last (the same in every leg)


def oracle_sample(w: gen.Workload, n_qblocks: int = ORACLE_QBLOCKS):
    """Time the CPU oracle, as it stands, on a bounded sample of one layer call of the workload and scale to a
    step.  Returns (frames_per_s, description, threads, parts)."""
    from oracle import hybrid_attention as oa
    f64 = gen.bf16_bits_to_f64
    Wb, bb = gen.merge_weights(w, 0)
    st = oa.HybridStream(w.batch, w.heads, w.head_dim, w.block, w.past_chunks, topk=w.topk,
                         keep_permille=w.keep_permille, W=f64(Wb), bias=f64(bb), eps=w.eps)
    for c in range(w.past_chunks):       # fill the window (no eviction yet: untimed)
        kc, vc = gen.clean_kv(w, 0, c)
        st.append(f64(kc), f64(vc))
    kc, vc = gen.clean_kv(w, 0, w.past_chunks)
    kc, vc = f64(kc), f64(vc)
    t0 = time.perf_counter()
    st.append(kc, vc)                     # one eviction + absorb + append, whole layer
    t_append = time.perf_counter() - t0
    q, k, v = (f64(t) for t in gen.qkv(w, 0, w.past_chunks + 1, 0))
    t0 = time.perf_counter()
    mask, _ = st.select(q, k)
    t_select = time.perf_counter() - t0
    tm = mask.shape[2]
    qbl = sorted(set(int(x) for x in np.linspace(0, tm - 1, n_qblocks)))
    t0 = time.perf_counter()
    st.forward(q, k, v, mask=mask, q_blocks=qbl)      # sparse attention on the sample + full history read-out
    t_fwd_sample = time.perf_counter() - t0
    rows = sum(min(w.block, w.chunk_tokens - i * w.block) for i in qbl)
    t_forward = t_select + t_fwd_sample * (w.chunk_tokens / rows)
    t_step = w.layers * (w.steps * t_forward + t_append)
    desc = (f"1 of {w.layers} layers: append+absorb of one chunk (all heads), selection (all heads), attention on "
            f"query blocks {qbl} of {tm} (all heads) scaled by rows; step = layers*(steps*forward+append)")
    try:
        import threadpoolctl
        thr = max([p["num_threads"] for p in threadpoolctl.threadpool_info()] or [1])
    except Exception:
        thr = os.cpu_count() or 1
    return w.chunk_frames / t_step, desc, thr, {"t_forward_s": t_forward, "t_append_s": t_append}


def oracle_baseline(w: gen.Workload, repeats: int = 3):
    """The cpu_baseline object: `repeats` runs of the same sample, harmonic mean, with the spread."""
    vals = []
    for _ in range(repeats):
        fps, desc, thr, _ = oracle_sample(w)
        vals.append(fps)
    value = len(vals) / sum(1.0 / x for x in vals)
    return {"value": value, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc, "repeats": repeats,
            "min": min(vals), "max": max(vals)}


def config_of(w: gen.Workload, swa_kernel):
    return {"workload": w.name, "layers": w.layers, "denoise_steps": w.steps, "batch": w.batch, "heads": w.heads,
            "head_dim": w.head_dim, "chunk_tokens": w.chunk_tokens, "window_frames": w.window_frames,
            "block": w.block, "keep_permille": w.keep_permille,
            "l2": "inputs larger than L2 (distinct q/k/v per layer, 1.3 GB per pass; caches 5.2 GB)",
            "swa_kernel": swa_kernel}


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for i in range(args.warmup + args.steps):
        fps, desc, thr, _ = oracle_sample(w)
        if i >= args.warmup:
            vals.append(fps)
    value = len(vals) / sum(1.0 / v for v in vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * w.chunk_frames / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w, "tcgen05"),       # the configuration of the arm it is compared with
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc,
                             "repeats": len(vals), "min": min(vals), "max": max(vals)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------- our arm
def kept_flops(mask_bool: np.ndarray, w: gen.Workload) -> float:
    """Algorithmic FLOPs of the sparse attention for a selection: 4 d sum_i rows_i sum_{j kept} cols_j (unpadded)."""
    nb = w.blocks_per_chunk
    sizes = np.array([min(w.block, w.chunk_tokens - i * w.block) for i in range(nb)], dtype=np.float64)
    cols = np.tile(sizes, mask_bool.shape[-1] // nb)
    kept_cols = (mask_bool * cols).sum(axis=-1)              # [B,H,Tm]
    return float(4.0 * w.head_dim * (kept_cols * sizes).sum())


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2604_10103_b200 import binding as hf, build as hfbuild

    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    if rank == 0:
        hfbuild.build()
    if world > 1:
        dist.barrier()
    peaks = load_peaks()
    ctx = hf.Context(hf.make_config(w), device=local)
    L, P = w.layers, w.past_chunks
    shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)
    g = torch.Generator(device="cuda"); g.manual_seed(replicas.replica_seed(1234, rank))
    rn = lambda: torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    q = [rn() for _ in range(L)]; k = [rn() for _ in range(L)]; v = [rn() for _ in range(L)]
    kc = [rn() for _ in range(L)]; vc = [rn() for _ in range(L)]
    o = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    for l in range(L):
        Wb, bb = gen.merge_weights(w, l)
        ctx.hf_set_merge_weights(l, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
        for c in range(P + 1):                       # fill the window and evict once: steady state
            ctx.hf_kv_append(l, kc[(l + c) % L], vc[(l + c) % L])
    torch.cuda.synchronize()

    def step():
        # Alg. 2 for one chunk: the denoising steps of every layer, then the clean chunk of every layer is committed
        # (all layers evict at that same moment: one layer-batched call)
        for l in range(L):
            for s in range(w.steps):
                ctx.hf_hybrid_forward(l, q[(l + s) % L], k[(l + s) % L], v[(l + s) % L], o)
        if args.per_layer_commit:
            for l in range(L):
                ctx.hf_kv_append(l, kc[l], vc[l])
        else:
            ctx.hf_kv_append_layers(0, kc, vc)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = ctx.hf_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    launches = ctx.hf_launch_count() - n0
    # One more step straight after the timed ones (same clocks, same power state), with an event at every call boundary:
    # where the step's time goes, call by call, and what is left between the calls.
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(L * w.steps + 2)]
    if not args.no_extras:
        i = 0
        for l in range(L):
            for s_ in range(w.steps):
                marks[i].record(); i += 1
                ctx.hf_hybrid_forward(l, q[(l + s_) % L], k[(l + s_) % L], v[(l + s_) % L], o)
        marks[i].record(); i += 1
        if args.per_layer_commit:
            for l in range(L):
                ctx.hf_kv_append(l, kc[l], vc[l])
        else:
            ctx.hf_kv_append_layers(0, kc, vc)
        marks[i].record()
    barrier()
    ms = e0.elapsed_time(e1)
    breakdown = None
    if not args.no_extras:
        fw = [marks[j].elapsed_time(marks[j + 1]) * 1e3 for j in range(L * w.steps)]
        commit_us = marks[L * w.steps].elapsed_time(marks[L * w.steps + 1]) * 1e3
        breakdown = {"forward_us_mean": statistics.mean(fw), "forward_us_min": min(fw), "forward_us_max": max(fw),
                     "forwards_ms": sum(fw) / 1e3, "commit_us": commit_us, "step_ms": marks[0].elapsed_time(marks[-1]),
                     "note": "one step run directly after the timed steps with a CUDA event at every call boundary; "
                             "forward = pooling + selection + attention (history term inside), commit = the layer-batched "
                             "cache commit (state update of 30 evicted chunks + copy and pooling of 30 new ones)"}
    clocks = sampler.stop() if rank == 0 else None
    ms, frames = replicas.aggregate(ms, args.steps * w.chunk_frames * w.batch)     # slowest rank, frames of all ranks
    ms_per_step = ms / args.steps
    value = replicas.throughput(frames, ms)

    # ---- per-stage split and the dominant kernel's launch time (CUDA events around batches of single-stage calls)
    def timed(fn, reps):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for r in range(reps):
            fn(r)
        b.record(); torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e3      # us per call

    stage = {}
    roof = None
    if args.no_extras:      # profiling runs: only the step loop above
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "warmup": args.warmup, "ms_per_step": ms_per_step, "gpu_launches": int(launches),
                              "config": {"workload": w.name, "layers": w.layers}, "extras": "skipped"}))
        ctx.close()
        if world > 1:
            dist.destroy_process_group()
        return
    if rank == 0:
        # The kernel-alone figures below are burst measurements (batches of a few milliseconds each): one second of idle
        # first, so that the board's power controller, which the step loop above has driven towards its cap, starts from rest
        time.sleep(1.0)
        reps = 2 * L
        stage["select_us"] = timed(lambda r: ctx.hf_block_select(r % L, q[r % L], k[r % L]), reps)
        for l in range(L):
            ctx.hf_block_select(l, q[l], k[l])
        stage["sparse_swa_us"] = timed(lambda r: ctx.hf_sparse_swa(r % L, q[r % L], k[r % L], v[r % L], o), reps)
        # the kernel the step loop launches: sparse attention with the history term formed inside (one launch per call)
        stage["swa_merged_us"] = timed(lambda r: ctx.hf_sparse_swa_merged(r % L, q[r % L], k[r % L], v[r % L], o), reps)
        # the backward kernels of the sparse branch (layer 0's selection; lse from its forward), timed alone
        lse = torch.empty(shape[:3], dtype=torch.float32, device="cuda")
        g_out = torch.randn(shape, device="cuda").to(torch.bfloat16); dq_ = torch.empty_like(o); dk_ = torch.empty_like(o); dv_ = torch.empty_like(o)
        ctx.hf_sparse_swa(0, q[0], k[0], v[0], o, lse=lse)
        o_fwd = o.clone()
        stage["backward_dq_us"] = timed(lambda r: ctx.hf_sparse_swa_backward_dq(0, q[0], k[0], v[0], o_fwd, lse, g_out, dq_), 16)
        stage["backward_dkv_us"] = timed(lambda r: ctx.hf_sparse_swa_backward_dkv(0, q[0], k[0], v[0], o_fwd, lse, g_out, dk_, dv_), 16)
        stage["backward_dq_history_us"] = timed(lambda r: ctx.hf_linear_attn_backward_dq(0, q[0], g_out, dq_), 16)
        del g_out, dq_, dk_, dv_, o_fwd
        stage["linear_us"] = timed(lambda r: ctx.hf_linear_attn(r % L, q[r % L], o), reps)
        stage["forward_us"] = timed(lambda r: ctx.hf_hybrid_forward(r % L, q[r % L], k[r % L], v[r % L], o), reps)
        stage["absorb_us"] = timed(lambda r: ctx.hf_state_absorb(r % L, kc[r % L], vc[r % L], w.chunk_tokens), reps)
        stage["append_with_absorb_us"] = timed(lambda r: ctx.hf_kv_append(r % L, kc[r % L], vc[r % L]), reps)
        # the same two stages for all layers in one call (what the step loop uses)
        kc_all = torch.stack(kc); vc_all = torch.stack(vc)
        stage["absorb_layers_us"] = timed(lambda r: ctx.hf_state_absorb_layers(0, L, kc_all, vc_all, w.chunk_tokens), 6)
        stage["append_layers_us"] = timed(lambda r: ctx.hf_kv_append_layers(0, kc, vc), 6)
        del kc_all, vc_all
        # algorithmic work of one sparse-SWA launch, from the actual selection of layer 0
        tn = ctx.hf_query(0, hf.HF_Q_KEY_BLOCKS); tm = ctx.hf_query(0, hf.HF_Q_QUERY_BLOCKS); mw = ctx.hf_query(0, hf.HF_Q_MASK_WORDS)
        mask = torch.zeros((w.batch, w.heads, tm, mw), dtype=torch.int32, device="cuda")
        ctx.hf_block_select(0, q[0], k[0], mask)
        torch.cuda.synchronize()
        flops_swa = kept_flops(hf.unpack_mask(mask.cpu().numpy().view(np.uint32), tn), w)
        flops_hist = 2.0 * w.head_dim * w.head_dim * w.batch * w.heads * w.chunk_tokens      # phi(Q) S of Eq. 4, once
        flops = flops_swa + flops_hist
        ach = flops / (stage["swa_merged_us"] * 1e-6) / 1e12
        # the kernel is timed alone in a loop of a few milliseconds: the burst figure is the denominator that applies
        peak = peaks["bf16_tflops"]
        ach_loop = flops / (breakdown["forward_us_mean"] * 1e-6) / 1e12 if breakdown else None
        roof = {"bound": "tensor", "kernel": "k_swa_tc5 with the history term inside (hf_sparse_swa_merged)", "achieved": ach, "peak": peak,
                "unit": "TFLOP/s", "frac": ach / peak,
                "peak_source": f"{peaks['source']} (burst cuBLAS bf16: the kernel is timed alone over {reps} launches after 1 s of idle; sustained {peaks['bf16_tflops_sustained']})",
                "frac_of_sustained": ach / peaks["bf16_tflops_sustained"], "frac_of_datasheet_2250": ach / 2250.0,
                # the whole forward (pooling + selection + attention) inside the seconds-long step loop, same FLOPs, against the sustained figure
                "forward_in_step_loop_tflops": ach_loop,
                "forward_in_step_loop_frac_of_sustained": ach_loop / peaks["bf16_tflops_sustained"] if ach_loop else None,
                "flops_per_launch": flops, "flops_kept_tiles": flops_swa, "flops_history": flops_hist,
                "attention_alone_tflops": flops_swa / (stage["sparse_swa_us"] * 1e-6) / 1e12,
                "traffic": SWA_DRAM_BYTES_PER_LAUNCH}
        # backward: 6 d FLOP per (query row, kept key) pair for dq (S, dP, dQ); 8 d per pair with the key in the CURRENT chunk
        # for dk / dv (S^T, dP^T, dV, dK)
        m_bool = hf.unpack_mask(mask.cpu().numpy().view(np.uint32), tn)
        m_cur = np.zeros_like(m_bool); m_cur[..., tn - w.blocks_per_chunk:] = m_bool[..., tn - w.blocks_per_chunk:]
        stage["backward_dq_tflops"] = 1.5 * flops_swa / (stage["backward_dq_us"] * 1e-6) / 1e12
        stage["backward_dkv_tflops"] = 2.0 * kept_flops(m_cur, w) / (stage["backward_dkv_us"] * 1e-6) / 1e12
        bytes_absorb = 2 * w.batch * w.heads * w.chunk_tokens * w.head_dim * 2
        stage["absorb_gbs"] = bytes_absorb / (stage["absorb_us"] * 1e-6) / 1e9
        stage["absorb_frac_hbm"] = stage["absorb_gbs"] / peaks["hbm_gbs"]
        stage["append_gbs"] = 3 * bytes_absorb / (stage["append_with_absorb_us"] * 1e-6) / 1e9   # absorb read + copy read + write
        stage["append_frac_hbm"] = stage["append_gbs"] / peaks["hbm_gbs"]
        stage["absorb_layers_gbs"] = L * bytes_absorb / (stage["absorb_layers_us"] * 1e-6) / 1e9
        stage["absorb_layers_frac_hbm"] = stage["absorb_layers_gbs"] / peaks["hbm_gbs"]
        stage["append_layers_gbs"] = L * 3 * bytes_absorb / (stage["append_layers_us"] * 1e-6) / 1e9
        stage["append_layers_frac_hbm"] = stage["append_layers_gbs"] / peaks["hbm_gbs"]

    # ---- the paper's isolating contrast (its Tab. 3, whole-model FPS there), attention only here: dense short-window
    # attention and dense window-21 attention (every block kept, no linear branch needed) against the hybrid forward
    contrast = None
    if rank == 0:
        contrast = {"hybrid_w9_forward_us": stage["forward_us"]}
        for name, win in (("dense_w9_swa_us", w.window_frames), ("dense_w21_swa_us", 21)):
            wd = w.with_(layers=1, window_frames=win, keep_permille=1000, topk=0)
            cd = hf.Context(hf.make_config(wd), device=local)
            for c_ in range(wd.past_chunks):
                cd.hf_kv_append(0, kc[c_ % L], vc[c_ % L])
            cd.hf_block_select(0, q[0], k[0])
            contrast[name] = timed(lambda r: cd.hf_sparse_swa(0, q[r % L], k[r % L], v[r % L], o), 8)
            cd.close()
        contrast["note"] = ("one layer call, 4680 queries; dense = all key blocks kept (111 at window 9, 259 at window 21); the "
                            "paper reports 21.8 -> 29.5 whole-model FPS for dense window 9 -> hybrid and 15.4 for dense window 21")

    # ---- the one-matrix reading of the history branch's Linear: read-out + projection over all heads + attention
    if rank == 0:
        wf = w.with_(layers=1)
        cf = hf.Context(hf.make_config(wf, merge=hf.HF_MERGE_FULL_WIDTH), device=local)
        Wfb, bfb = gen.merge_weights_full(wf, 0)
        cf.hf_set_merge_weights(0, hf.bits_to_cuda(Wfb), hf.bits_to_cuda(bfb))
        for c_ in range(wf.past_chunks + 1):
            cf.hf_kv_append(0, kc[c_ % L], vc[c_ % L])
        t_lin = timed(lambda r: cf.hf_linear_attn(0, q[r % L], o), 16)
        t_fwd = timed(lambda r: cf.hf_hybrid_forward(0, q[r % L], k[r % L], v[r % L], o), 16)
        hd = wf.heads * wf.head_dim
        contrast["full_width_merge"] = {"linear_us": t_lin, "forward_us": t_fwd,
                                        "projection_gflop": 2.0 * wf.batch * wf.chunk_tokens * hd * hd / 1e9,
                                        "note": "history branch with one [H d, H d] projection over all heads: read-out kernel + projection kernel"
                                                " (bf16 hi/lo operand, tcgen05), then the attention kernel adds the term"}
        cf.close()

    # ---- end to end through the host-buffer entry points (H2D of q,k,v and D2H of o inside the timed region)
    e2e = None
    e2e_steps = max(1, min(args.steps, 2))
    hq, hk, hv, ho = (torch.empty(shape, dtype=torch.bfloat16).pin_memory() for _ in range(4))
    hq.copy_(q[0].cpu()); hk.copy_(k[0].cpu()); hv.copy_(v[0].cpu())

    def step_host():
        for l in range(L):
            for s in range(w.steps):
                ctx.hf_hybrid_forward_host(l, hq, hk, hv, ho)
            ctx.hf_kv_append_host(l, hk, hv)

    step_host()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_host()
    barrier()
    t_e2e = time.perf_counter() - t0
    t_e2e_ms, frames_e2e = replicas.aggregate(t_e2e * 1e3, e2e_steps * w.chunk_frames * w.batch)
    nbytes = hq.numel() * 2
    e2e = {"value": replicas.throughput(frames_e2e, t_e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": L * (w.steps * 3 + 2) * nbytes, "d2h_bytes_per_step": L * w.steps * nbytes, "steps": e2e_steps}
    flags, detail = ctx.hf_get_device_status()

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic",
                "config": config_of(w, {1: "mma.sync", 2: "tcgen05"}.get(ctx.hf_query(0, hf.HF_Q_SWA_KERNEL))),
                "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e, "roofline": roof, "stages": stage,
                "step_breakdown": breakdown, "contrast": contrast,
                "cpu_baseline": oracle_baseline(w),
                "context": {"paper_end_to_end_fps_h100": 29.5, "note": "whole model, video frames/s; not this metric"}}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Stage times and roofline fractions over the grid keep in {10,25,50,100} % x window in {3,9,21} frames x head_dim
    in {64,128} x block in {64,128} x batch in {1,4} at 1560 tokens per latent frame, 12 heads, 3-frame chunks: one JSON
    line per grid point (layer calls rotate over several layer contexts so that the inputs exceed L2)."""
    import torch
    from paper_2604_10103_b200 import binding as hf, build as hfbuild
    hfbuild.build()
    torch.cuda.set_device(0)
    peaks = load_peaks()
    out = open(args.sweep_out, "w") if args.sweep_out else sys.stdout

    def timed(fn, reps):
        for r in range(3):
            fn(r)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for r in range(reps):
            fn(r)
        b.record(); torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e3

    for batch in (1, 4):
        for d in (64, 128):
            for blk in (64, 128):
                for win in (3, 9, 21):
                    for permille in (100, 250, 500, 1000):
                        L = 4 if batch == 1 else 2
                        w = gen.layer_832x480().with_(name="sweep", batch=batch, head_dim=d, block=blk, window_frames=win,
                                                      keep_permille=permille, topk=0, layers=L)
                        ctx = hf.Context(hf.make_config(w))
                        shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)
                        g = torch.Generator(device="cuda"); g.manual_seed(4321)
                        rn = lambda: torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
                        q = [rn() for _ in range(L)]; k = [rn() for _ in range(L)]; v = [rn() for _ in range(L)]
                        o = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
                        for l in range(L):
                            Wb, bb = gen.merge_weights(w, l)
                            ctx.hf_set_merge_weights(l, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
                            for c in range(w.past_chunks + 1):
                                ctx.hf_kv_append(l, k[(l + c) % L], v[(l + c) % L])
                        reps = 4 * L
                        st = {"select_us": timed(lambda r: ctx.hf_block_select(r % L, q[r % L], k[r % L]), reps)}
                        st["sparse_swa_us"] = timed(lambda r: ctx.hf_sparse_swa(r % L, q[r % L], k[r % L], v[r % L], o), reps)
                        st["linear_us"] = timed(lambda r: ctx.hf_linear_attn(r % L, q[r % L], o), reps)
                        st["forward_us"] = timed(lambda r: ctx.hf_hybrid_forward(r % L, q[r % L], k[r % L], v[r % L], o), reps)
                        st["absorb_us"] = timed(lambda r: ctx.hf_state_absorb(r % L, k[r % L], v[r % L], w.chunk_tokens), reps)
                        st["append_us"] = timed(lambda r: ctx.hf_kv_append(r % L, k[r % L], v[r % L]), reps)
                        tn = ctx.hf_query(0, hf.HF_Q_KEY_BLOCKS); tm = ctx.hf_query(0, hf.HF_Q_QUERY_BLOCKS)
                        mw = ctx.hf_query(0, hf.HF_Q_MASK_WORDS)
                        mask = torch.zeros((w.batch, w.heads, tm, mw), dtype=torch.int32, device="cuda")
                        ctx.hf_block_select(0, q[0], k[0], mask)
                        torch.cuda.synchronize()
                        flops = kept_flops(hf.unpack_mask(mask.cpu().numpy().view(np.uint32), tn), w)
                        tf = flops / (st["sparse_swa_us"] * 1e-6) / 1e12
                        nbytes = 2 * w.batch * w.heads * w.chunk_tokens * w.head_dim * 2
                        flags, _ = ctx.hf_get_device_status()
                        line = {"batch": batch, "head_dim": d, "block": blk, "window_frames": win, "keep_permille": permille,
                                "key_blocks": tn, "kept_blocks": ctx.hf_query(0, hf.HF_Q_KEPT_BLOCKS),
                                "swa_kernel": {1: "mma.sync", 2: "tcgen05", 3: "tcgen05 ping-pong"}.get(ctx.hf_query(0, hf.HF_Q_SWA_KERNEL)),
                                **{k_: round(v_, 2) for k_, v_ in st.items()},
                                "swa_tflops": round(tf, 1), "swa_frac_of_burst_peak": round(tf / peaks["bf16_tflops"], 3),
                                "absorb_frac_hbm": round(nbytes / (st["absorb_us"] * 1e-6) / 1e9 / peaks["hbm_gbs"], 3),
                                "append_frac_hbm": round((3 * nbytes if w.past_chunks else nbytes) / (st["append_us"] * 1e-6) / 1e9 / peaks["hbm_gbs"], 3),
                                "device_status": flags}
                        out.write(json.dumps(line) + "\n"); out.flush()
                        ctx.close()
                        del q, k, v, o
                        torch.cuda.empty_cache()
    if out is not sys.stdout:
        out.close()


def run_profile_backward():
    """A small stand-alone run of the backward kernels, for profilers: one layer of the 832x480 shape (window 9, two cached
    chunks and one absorbed), three calls of each of dq, dk / dv and the read-out's dq."""
    import torch
    from paper_2604_10103_b200 import binding as hf, build as hfbuild
    hfbuild.build()
    w = gen.layer_832x480().with_(layers=1)
    ctx = hf.Context(hf.make_config(w))
    Wb, bb = gen.merge_weights(w, 0)
    ctx.hf_set_merge_weights(0, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
    g = torch.Generator(device="cuda"); g.manual_seed(98)
    shape = (w.batch, w.heads, w.chunk_tokens, w.head_dim)
    mk = lambda: torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    for _ in range(w.past_chunks + 1):
        ctx.hf_kv_append(0, mk(), mk())
    q, k, v, go = mk(), mk(), mk(), mk()
    o = torch.empty_like(q); dq = torch.empty_like(q); dk = torch.empty_like(q); dv = torch.empty_like(q)
    lse = torch.empty(shape[:3], dtype=torch.float32, device="cuda")
    ctx.hf_block_select(0, q, k)
    ctx.hf_sparse_swa(0, q, k, v, o, lse=lse)
    out = {"stage": "backward"}
    for name, fn in (("dq_us", lambda: ctx.hf_sparse_swa_backward_dq(0, q, k, v, o, lse, go, dq)),
                     ("dkv_us", lambda: ctx.hf_sparse_swa_backward_dkv(0, q, k, v, o, lse, go, dk, dv)),
                     ("dq_history_us", lambda: ctx.hf_linear_attn_backward_dq(0, q, go, dq))):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(3):
            if i == 2:
                a.record()
            fn()
        b.record(); torch.cuda.synchronize()
        out[name] = a.elapsed_time(b) * 1e3
    out["status"] = ctx.hf_get_device_status()
    print(json.dumps(out))
    ctx.close()


def run_profile_stage(args):
    """A small stand-alone run of one stage, for profilers: the layer-batched state update on 13 layers of the
    832x480 layer shape (156 (layer, head) items, under 1 GB on the device; no cache ring is allocated)."""
    import torch
    from paper_2604_10103_b200 import binding as hf, build as hfbuild
    if args.profile_stage == "backward":
        return run_profile_backward()
    hfbuild.build()
    L = 13
    w = gen.layer_832x480().with_(layers=L, window_frames=3)        # window == chunk: no ring
    ctx = hf.Context(hf.make_config(w))
    for l in range(L):
        Wb, bb = gen.merge_weights(w, l)
        ctx.hf_set_merge_weights(l, hf.bits_to_cuda(Wb), hf.bits_to_cuda(bb))
    g = torch.Generator(device="cuda"); g.manual_seed(99)
    shape = (L, w.batch, w.heads, w.chunk_tokens, w.head_dim)
    k = torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn(shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        if i == 2:
            a.record()
        ctx.hf_state_absorb_layers(0, L, k, v, w.chunk_tokens)
    b.record(); torch.cuda.synchronize()
    nbytes = 2 * k.numel() * 2
    us = a.elapsed_time(b) * 1e3
    print(json.dumps({"stage": "absorb_layers", "layers": L, "us": us, "gbs": nbytes / (us * 1e-6) / 1e9, "status": ctx.hf_get_device_status()}))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=30)
    ap.add_argument("--denoise-steps", type=int, default=4)
    ap.add_argument("--per-layer-commit", action="store_true",
                    help="commit the clean chunk layer by layer (hf_kv_append) instead of with one layer-batched call")
    ap.add_argument("--no-extras", action="store_true",
                    help="run only the warm-up and the timed step loop (no stage split, end-to-end leg or CPU baseline): "
                         "the command profilers are pointed at")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark line: per-stage times over the keep x window x head_dim x block x batch grid, "
                         "one JSON line per point (1 GPU)")
    ap.add_argument("--sweep-out", default=None, help="file for the sweep's JSON lines (default: stdout)")
    ap.add_argument("--profile-stage", default=None, choices=["absorb_layers", "backward"],
                    help="instead of the benchmark line: a small run of one stage alone (for ncu captures)")
    args = ap.parse_args()
    w = gen.full_depth_832x480(layers=args.layers, steps=args.denoise_steps)
    if args.profile_stage:
        run_profile_stage(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
