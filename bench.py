#!/usr/bin/env python
"""Benchmark of the copy-and-verify decode step (CopySpec, arXiv 2502.08923) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole hot path for one batch: suffix-match search, draft
gather, one verification forward of the 8B-class model over the (k+1)-row block against
the bf16 KV cache, LM-head argmax, prefix acceptance, KV truncation and the append to the
history - i.e. one replay of the generation loop's step graph.  The workload is the
8B-class verify configuration: batch 1, KV cache starting at 4,096 positions, gamma = 3,
k = 10, scripted-target mode with the accepted prefix uniform in [0, 10]; every input is
seeded and synthetic (random-init bf16 weights, N(0,1) KV fill, token paths built so that
each step accepts a prescribed number of draft tokens).

`value` is emitted tokens per second (accepted draft tokens plus the one guaranteed token
per step) with everything resident in HBM; `e2e` drives the same steps from pinned host
buffers through cs_step_host (one C call per step: copies in, search, verify, copies out,
host append), all inside the timed region.
With N > 1 every rank runs an independent replica (the path does not shard).
`--impl reference` times the CPU oracle, as it stands, on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "accepted tokens/sec"
UNIT = "tokens/s"
GAMMA, K_DRAFT, KV_START = 3, 10, 4096
WORKLOAD = "verify_8b_b1_kv4096_k10_scripted_tau_uniform"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from the
# committed ncu capture (profiles/); None until a capture of the current kernel exists.
NCU_TRAFFIC_BYTES_PER_LAUNCH = 111.8e6   # profiles/k_gemm_tc_verify8b_2layer_ncu_full.md


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def _taus(n_steps, seed=0):
    """Accepted prefix per step: uniform over 0..k, each value equally often."""
    rng = np.random.default_rng(seed)
    reps = -(-n_steps // (K_DRAFT + 1))
    return [int(t) for t in rng.permutation(np.repeat(np.arange(K_DRAFT + 1), reps))[:n_steps]]


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(names, f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def _dist():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# --------------------------------------------------------------------- CPU oracle leg
def oracle_sample(cfg8b, weights_cpu_layer0, kv_layer0, lm_head_cpu, hist, script, taus, n_steps, warmup):
    """Times the oracle, as it stands, on a bounded sample of the workload: the verification
    forward of ONE of the 32 decoder layers (block of k+1 rows against 4,096 cached
    positions) per step plus the search and acceptance, and the LM head once; the full
    step time is extrapolated as 32 * layer + LM head.  Returns tokens/s and details."""
    from oracle import copyspec_oracle as O
    from paper_2502_08923_b200 import inputs
    import threadpoolctl
    cfg1 = inputs.sliced(cfg8b, 1)
    h = [int(t) for t in hist]
    n = len(h)
    p0 = O.find_match(np.asarray(h), n, GAMMA, O.LATEST)
    draft = O.gather_draft(h, n, p0, GAMMA, K_DRAFT)
    block = [h[-1]] + draft
    # the forward only needs the embedding rows of the block's tokens: a small table of
    # those rows (taken from the LM-head matrix, which has the same shape and statistics)
    emb_small = lm_head_cpu[np.asarray(block, dtype=np.int64)]
    w = {"embed": emb_small, "lm_head": lm_head_cpu, "final_norm": weights_cpu_layer0["final_norm"],
         "layers": [weights_cpu_layer0["layer"]]}
    model = O.Model(cfg1, w, contract=True, cache_weights=True)
    cache = O.KVCache(cfg1, 1, KV_START + 64, dtype=np.float32)
    cache.a[0, :, 0, :, :KV_START, :] = kv_layer0
    rows = list(range(len(block)))
    t0 = time.perf_counter()
    logits, hidden = model.forward_block(rows, KV_START, cache, 0, return_hidden=True)
    t_first = time.perf_counter() - t0
    # LM head (final norm, logits, greedy token per row), weights already converted
    t0 = time.perf_counter()
    xn = O.rmsnorm(hidden, model._w(None, "final_norm"), cfg1.rms_eps)
    lg = model._mm(xn, None, "lm_head")
    am = [O.argmax_lowest(lg[r]) for r in range(len(block))]
    t_lm = time.perf_counter() - t0
    # per-step sample: search + one layer's forward + acceptance (an 8-row stand-in head)
    model._cache[(None, "lm_head")] = model._cache[(None, "lm_head")][:8]
    times = []
    for i in range(warmup + n_steps):
        t0 = time.perf_counter()
        p0 = O.find_match(np.asarray(h), n, GAMMA, O.LATEST)
        draft = O.gather_draft(h, n, p0, GAMMA, K_DRAFT)
        model.forward_block(rows, KV_START, cache, 0)
        O.accept_length(draft, [int(t) for t in script[:len(draft) + 1]])
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    t_layer = float(np.mean(times))
    step_s = cfg8b.n_layers * t_layer + t_lm
    tokens_per_step = float(np.mean([t + 1 for t in taus]))
    cores = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    return {"value": tokens_per_step / step_s, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": (f"{n_steps} steps of search + one decoder layer (of 32) over an 11-row block and 4,096 cached "
                       f"positions + acceptance ({t_layer * 1e3:.1f} ms each), LM head once ({t_lm * 1e3:.0f} ms); "
                       f"step time extrapolated as 32 x layer + LM head = {step_s * 1e3:.0f} ms"),
            "ms_per_step": step_s * 1e3, "first_call_s": t_first}


def _oracle_inputs(cfg, seed=0):
    """The slices the CPU sample needs, drawn on the CPU with the bench's recipe."""
    import torch
    from paper_2502_08923_b200 import inputs
    g = torch.Generator().manual_seed(seed)

    def normal(*shape):
        return torch.empty(*shape, dtype=torch.float32).normal_(0.0, 0.02, generator=g).to(torch.bfloat16)

    d, f = cfg.d_model, cfg.d_ffn
    layer = {"attn_norm": torch.ones(d, dtype=torch.bfloat16), "wqkv": normal(cfg.qkv_dim, d),
             "wo": normal(d, cfg.q_dim), "ffn_norm": torch.ones(d, dtype=torch.bfloat16),
             "w_gate_up": normal(2 * f, d), "w_down": normal(d, f)}
    lm = normal(cfg.vocab, d)
    kv = torch.empty(2, cfg.n_kv_heads, KV_START, cfg.head_dim).normal_(0.0, 1.0, generator=g).to(torch.bfloat16)
    return {"layer": layer, "final_norm": torch.ones(d, dtype=torch.bfloat16)}, kv.float().numpy(), lm


def run_reference(args):
    rank, world, _ = _dist()
    if rank != 0:
        return 0
    from paper_2502_08923_b200 import inputs
    cfg = inputs.LLAMA8B
    steps = args.steps
    taus = _taus(args.warmup + steps)
    hist, script = inputs.tau_controlled_case(np.random.default_rng(0), taus, GAMMA, K_DRAFT, KV_START, cfg.vocab)
    w0, kv0, lm = _oracle_inputs(cfg)
    res = oracle_sample(cfg, w0, kv0, lm, hist, script, taus, steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "gamma": GAMMA, "k": K_DRAFT, "batch": 1, "kv_start": KV_START},
            "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": res["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


def aggregate_replicas(ms_local, emitted_local, world, device):
    """Replicas share nothing: the job's time is the slowest rank's, its tokens the sum over
    ranks.  Returns (ms, tokens per second of the whole job)."""
    import torch
    import torch.distributed as dist
    if world == 1:
        return ms_local, emitted_local / (ms_local * 1e-3)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([float(emitted_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item()) / (float(t.item()) * 1e-3)


# ------------------------------------------------------------------------ CUDA leg
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_08923_b200 import binding as cs, inputs

    rank, world, local = _dist()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    cfg = inputs.LLAMA8B if args.layers <= 0 else inputs.sliced(inputs.LLAMA8B, args.layers)
    W, K = args.warmup, args.steps
    taus = _taus(W + K)
    ctx_len = KV_START
    while True:
        try:
            hist, script = inputs.tau_controlled_case(np.random.default_rng(0), taus, GAMMA, K_DRAFT, ctx_len, cfg.vocab)
            break
        except ValueError:
            ctx_len += 1024            # more steps than the 4,096-token context has room for
    max_new = len(script)
    n0 = len(hist)
    stride = (n0 + max_new + 64 + 3) // 4 * 4
    max_seq = n0 + max_new + K_DRAFT + 64

    weights = inputs.make_weights(cfg, seed=0, device=str(dev))
    ctx = cs.Context(cfg, weights, max_seq=max_seq, max_batch=1, k_max=K_DRAFT)
    kv = inputs.synthetic_kv(cfg, 1, max_seq, n0 - 1, seed=1, device=str(dev))
    hist_h = np.zeros((1, stride), dtype=np.int32)
    hist_h[0, :n0] = hist
    hist_d = torch.from_numpy(hist_h).to(dev)
    len_d = torch.tensor([n0], dtype=torch.int32, device=dev)
    kvlen_d = torch.tensor([n0 - 1], dtype=torch.int32, device=dev)
    script_d = torch.from_numpy(script[None, :].copy()).to(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident loop: W warm-up steps, then exactly K timed steps ------------
    ctx.cs_loop_begin(hist_d, len_d, kv, kvlen_d, GAMMA, K_DRAFT, max_new, script=script_d)
    launches_per_step = ctx.cs_loop_launches_per_step()
    ctx.cs_loop_steps(W)
    st0, _ = ctx.cs_loop_poll()
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ctx.cs_loop_steps(K)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    st1, done = ctx.cs_loop_poll()
    ctx.cs_loop_end()
    emitted = st1["emitted"] - st0["emitted"]
    steps_run = st1["steps"] - st0["steps"]
    expect = sum(t + 1 for t in taus[W:W + K])
    if steps_run != K or emitted != expect:
        raise RuntimeError(f"loop ran {steps_run} steps / {emitted} tokens, expected {K} / {expect}")
    ms, value = aggregate_replicas(ms, emitted, world, dev)

    # ---- end to end from pinned host buffers: one cs_step_host call per step (history, length
    # and script row host -> device, search + verify, accepted length and tokens device -> host,
    # the host appends)
    Ke = min(K, 50)
    hist_p = torch.from_numpy(hist_h.copy()).pin_memory()
    len_p = torch.tensor([n0], dtype=torch.int32).pin_memory()
    scr_p = torch.zeros(1, K_DRAFT + 1, dtype=torch.int32).pin_memory()
    acc_p = torch.zeros(1, dtype=torch.int32).pin_memory()
    out_p = torch.zeros(1, K_DRAFT + 1, dtype=torch.int32).pin_memory()
    hist_e = torch.empty_like(hist_d)
    len_e = torch.empty_like(len_d)
    kvlen_d.fill_(n0 - 1)
    script_pad = torch.from_numpy(np.concatenate([script, np.full(K_DRAFT + 1, -1, dtype=np.int32)]))
    d2h = (acc_p.numel() + out_p.numel()) * 4
    h2d_total = 0

    def host_step(n, e):
        nonlocal h2d_total
        scr_p[0].copy_(script_pad[e:e + K_DRAFT + 1])
        ctx.cs_step_host(hist_p, len_p, hist_e, len_e, kv, kvlen_d, GAMMA, K_DRAFT, acc_p, out_p, script_host=scr_p)
        h2d_total += n * 4 + 4 + scr_p.numel() * 4
        tau = int(acc_p[0])
        return n + tau + 1, e + tau + 1

    n, e = n0, 0
    for _ in range(3):
        n, e = host_step(n, e)
    barrier()
    t0 = time.perf_counter()
    e_start = e
    h2d_total = 0
    for _ in range(Ke):
        n, e = host_step(n, e)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if hist_p[0, n0:n].tolist() != script[:e].tolist():
        raise RuntimeError("host-driven steps did not reproduce the script")
    e2e_val = world * (e - e_start) / e2e_s

    # ---- roofline of the dominant kernel (the weight-streaming projection GEMM) ---------
    kvlen_d.fill_(n0 - 1)
    last = torch.tensor([int(hist[-1])], dtype=torch.int32, device=dev)
    dr = torch.from_numpy(script[None, :K_DRAFT].copy()).to(dev)
    dl = torch.full((1,), K_DRAFT, dtype=torch.int32, device=dev)
    fam_ms, fam_n = None, None
    for _ in range(3):
        kvlen_d.fill_(n0 - 1)
        fam_ms, fam_n = ctx.cs_profile_verify_step(last, dr, dl, kv, kvlen_d)
    layer_bytes = cfg.n_layers * cfg.params_per_layer() * 2
    gemm_launches = max(1, fam_n["gemm"])
    peak, peak_kind = _peaks()
    achieved = layer_bytes / gemm_launches / (fam_ms["gemm"] / gemm_launches * 1e-3) / 1e9
    step_bytes = cfg.streamed_params() * 2 + (n0 - 1 + 0.5 * emitted) * cfg.kv_bytes_per_token()
    step_gbs = step_bytes / (ms / K * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "k_gemm_tc (layer projections)", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind,
                "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH,
                "bytes_per_launch": layer_bytes / gemm_launches, "launches_per_step": gemm_launches,
                "family_ms_per_step": fam_ms,
                "step": {"algorithmic_gb": step_bytes / 1e9, "achieved_gbs": step_gbs, "frac_of_measured_copy": step_gbs / peak,
                         "frac_of_8tbs": step_gbs / 8000.0}}

    line = None
    if rank == 0:
        # ---- CPU oracle on the host cores, bounded sample (rank 0, N = 1 only) ---------
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            w0 = {"layer": {k2: v.cpu() for k2, v in weights["layers"][0].items()}, "final_norm": weights["final_norm"].cpu()}
            kv0 = kv[0, :, 0, :, :KV_START, :].float().cpu().numpy()
            res = oracle_sample(cfg, w0, kv0, weights["lm_head"].cpu(), hist, script, taus, 150, 3)
            cpu = {k2: res[k2] for k2 in ("value", "unit", "cores", "kind", "sample")}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "model_shape": f"{cfg.n_layers}L d4096 H32/8 Dh128 F14336 V128256", "batch": 1,
                           "gamma": GAMMA, "k": K_DRAFT, "kv_start": n0 - 1, "kv_end": n0 - 1 + st1["emitted"],
                           "tokens_per_step": emitted / K, "l2": "inputs larger than L2 (15 GB of weights per step)",
                           "replicas": world, "draft_tokens_accepted_per_s": world * (emitted - K) / (ms * 1e-3)},
                "clocks": clocks,
                "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d_total // Ke, "d2h_bytes_per_step": d2h,
                        "steps": Ke, "ms_per_step": e2e_s / Ke * 1e3},
                "gpu_launches": launches_per_step * K,
                "roofline": roofline, "cpu_baseline": cpu}
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0



# ------------------------------------------------------------- the other workloads
def run_workload(args):
    """Additional measurements (not the headline line): the long-context and multi-turn loops
    at full shape, plain one-token decoding from the same kernels, and the search alone."""
    import torch
    from paper_2502_08923_b200 import binding as cs, inputs
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    name = args.workload
    W, K = args.warmup, args.steps
    ev = lambda: torch.cuda.Event(enable_timing=True)
    if name == "match_search":
        hist, kinds, _ = inputs.match_search_histories()
        hd = torch.from_numpy(hist).to(dev)
        ld = torch.full((64,), 32768, dtype=torch.int32, device=dev)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        out = {}
        for gamma in (3, 5):
            bufs = cs.cs_find_match(hd, ld, gamma, K_DRAFT)
            for mode in ("warm", "cold"):
                ts = []
                for i in range(W + K):
                    if mode == "cold":
                        flush.fill_(i & 1)
                    e0, e1 = ev(), ev()
                    e0.record()
                    cs.cs_find_match(hd, ld, gamma, K_DRAFT, out=bufs)
                    e1.record()
                    torch.cuda.synchronize()
                    if i >= W:
                        ts.append(e0.elapsed_time(e1) * 1e3)
                out[f"gamma{gamma}_{mode}_us_per_batch"] = float(np.median(ts))
        # the gamma-gram index (Sec. 3.1) on the same batch: bulk build once, then one step's worth
        # of update (10 appended tokens per sequence) + lookup
        idx = cs.GramIndex(64, 32768, 3)
        ld0 = torch.full((64,), 32758, dtype=torch.int32, device=dev)
        e0, e1 = ev(), ev()
        e0.record(); idx.cs_gram_index_update(hd, ld0); e1.record(); torch.cuda.synchronize()
        out["index_build_us_per_batch"] = e0.elapsed_time(e1) * 1e3
        bufs = idx.cs_find_match_indexed(hd, ld, K_DRAFT)
        ts = []
        for i in range(W + K):
            flush.fill_(i & 1)
            e0, e1 = ev(), ev()
            e0.record()
            idx.cs_gram_index_update(hd, ld)
            idx.cs_find_match_indexed(hd, ld, K_DRAFT, out=bufs)
            e1.record()
            torch.cuda.synchronize()
            if i >= W:
                ts.append(e0.elapsed_time(e1) * 1e3)
        out["index_update_lookup_cold_us_per_batch"] = float(np.median(ts))
        # where the index pays: the same comparison on 8 histories of 262,144 tokens
        hist_l, _, _ = inputs.match_search_histories(batch=8, n=262144, n_spans=4, span_lo=64, span_hi=256)
        hl = torch.from_numpy(hist_l).to(dev)
        ll = torch.full((8,), 262144, dtype=torch.int32, device=dev)
        idx_l = cs.GramIndex(8, 262144, 3)
        idx_l.cs_gram_index_update(hl, torch.full((8,), 262134, dtype=torch.int32, device=dev))
        bs, bi = cs.cs_find_match(hl, ll, 3, K_DRAFT), idx_l.cs_find_match_indexed(hl, ll, K_DRAFT)
        t_scan, t_idx = [], []
        for i in range(W + K):
            flush.fill_(i & 1)
            e0, e1, e2 = ev(), ev(), ev()
            e0.record()
            cs.cs_find_match(hl, ll, 3, K_DRAFT, out=bs)
            e1.record()
            idx_l.cs_gram_index_update(hl, ll)
            idx_l.cs_find_match_indexed(hl, ll, K_DRAFT, out=bi)
            e2.record()
            torch.cuda.synchronize()
            if i >= W:
                t_scan.append(e0.elapsed_time(e1) * 1e3)
                t_idx.append(e1.elapsed_time(e2) * 1e3)
        if not all(torch.equal(x, y) for x, y in zip(bs, bi)):
            raise RuntimeError("index and scan disagree")
        out["long_8x262144_scan_cold_us"] = float(np.median(t_scan))
        out["long_8x262144_index_update_lookup_cold_us"] = float(np.median(t_idx))
        us = out["gamma3_cold_us_per_batch"]
        line = {"metric": "match-search us/seq", "value": us / 64, "unit": "us", "higher_is_better": False,
                "n_gpus": 1, "steps": K, "warmup": W, "dtype": "int32", "data": "synthetic",
                "config": {"workload": "match_search_64x32768_zipf", "k": K_DRAFT, "bytes_per_batch": 64 * 32768 * 4,
                           "gbs_cold": 64 * 32768 * 4 / us / 1e3, **out}}
        print(json.dumps(line), flush=True)
        return 0
    cfg = inputs.LLAMA8B
    if name == "prefill_b1_4096":
        # context ingestion through cs_prefill (chunks of 256 block rows through the same kernels)
        n_ctx = 4096
        weights = inputs.make_weights(cfg, seed=0, device=str(dev))
        ctx = cs.Context(cfg, weights, max_seq=n_ctx + 64, max_batch=1, k_max=K_DRAFT)
        kv = ctx.alloc_kv()
        hist = torch.from_numpy(inputs.zipf_tokens(np.random.default_rng(0), n_ctx, cfg.vocab, 1.1).astype(np.int32)[None, :]).to(dev)
        ld = torch.tensor([n_ctx], dtype=torch.int32, device=dev)
        kvl = torch.zeros(1, dtype=torch.int32, device=dev)
        ts = []
        for i in range(3 + min(K, 10)):
            e0, e1 = ev(), ev()
            e0.record()
            ctx.cs_prefill(hist, ld, n_ctx, kv, kvl)
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                ts.append(e0.elapsed_time(e1))
        ms = float(np.median(ts))
        flops = 2.0 * cfg.streamed_params() * n_ctx
        line = {"metric": "prefill tokens/sec", "value": n_ctx / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
                "steps": len(ts), "warmup": 3, "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": name, "batch": 1, "context": n_ctx, "chunk_rows": 256,
                           "weight_passes": n_ctx // 256, "dense_tflops": flops / (ms * 1e-3) / 1e12}}
        print(json.dumps(line), flush=True)
        ctx.close()
        return 0
    if name == "drafted_b1_k10":
        return run_drafted(args, cs, inputs, dev)
    if name == "long_context_b1_k10":
        cases, k = [inputs.long_context_case(100)], 10
    elif name == "long_context_b8_k20":
        cases, k = [inputs.long_context_case(100 + b) for b in range(8)], 20
    elif name == "multi_turn_b16_k10":
        cases, k = [inputs.multi_turn_case(200 + b)[:2] for b in range(16)], 10
    elif name == "k_sweep_long_context_b1":
        # a long script, so that even 101-token steps leave room for a representative stretch
        cases, k = [inputs.long_context_case(100, script_len=16384)], 100
    elif name == "verify_plain_decode":
        taus = _taus(W + K)
        cases, k = [inputs.tau_controlled_case(np.random.default_rng(0), taus, GAMMA, K_DRAFT, KV_START, cfg.vocab)], 10
    else:
        raise SystemExit(f"unknown workload {name}")
    B = len(cases)
    n0 = max(len(h) for h, _ in cases)
    max_new = min(len(s) for _, s in cases)
    stride = (n0 + max_new + 67) // 4 * 4
    max_seq = n0 + max_new + k + 64
    weights = inputs.make_weights(cfg, seed=0, device=str(dev))
    ctx = cs.Context(cfg, weights, max_seq=max_seq, max_batch=B, k_max=k)
    kv = torch.zeros(cfg.n_layers, 2, B, cfg.n_kv_heads, max_seq, cfg.head_dim, dtype=torch.bfloat16, device=dev)
    g = torch.Generator(device=dev); g.manual_seed(1)
    for layer in range(cfg.n_layers):
        kv[layer, :, :, :, :n0 - 1, :] = torch.randn(2, B, cfg.n_kv_heads, n0 - 1, cfg.head_dim, device=dev,
                                                      generator=g).to(torch.bfloat16)
    h = np.zeros((B, stride), dtype=np.int32)
    lens = np.array([len(hh) for hh, _ in cases], dtype=np.int32)
    for b, (hh, _) in enumerate(cases):
        h[b, :len(hh)] = hh
    script_d = torch.from_numpy(np.stack([s[:max_new] for _, s in cases]).astype(np.int32)).to(dev)
    res = {}
    sweep = (100, 50, 20, 10, 5, 0) if name == "k_sweep_long_context_b1" else ((k, 0) if name != "verify_plain_decode" else (0,))
    for kk in sweep:
        steps = K if kk else min(4 * K, max_new - W - 1)
        steps = min(steps, (max_new // (kk + 1)) - W - 1)
        hd, ld = torch.from_numpy(h).to(dev), torch.from_numpy(lens).to(dev)
        kvl = torch.from_numpy(lens - 1).to(dev)
        ctx.cs_loop_begin(hd, ld, kv, kvl, GAMMA, kk, max_new, script=script_d)
        ctx.cs_loop_steps(W)
        st0, _ = ctx.cs_loop_poll()
        e0, e1 = ev(), ev()
        e0.record()
        ctx.cs_loop_steps(steps)
        e1.record()
        torch.cuda.synchronize()
        st1, _ = ctx.cs_loop_poll()
        ctx.cs_loop_end()
        ms = e0.elapsed_time(e1)
        em = st1["emitted"] - st0["emitted"]
        att = max(1, st1["attempts"] - st0["attempts"])
        res[kk] = {"tokens_per_s": em / (ms * 1e-3), "ms_per_step": ms / steps, "steps": steps,
                   "tokens_per_step": em / steps / B, "mean_tau": (st1["accepted"] - st0["accepted"]) / att,
                   "copied_frac": (st1["accepted"] - st0["accepted"]) / max(1, em)}
    main = res[k] if k in res and name != "verify_plain_decode" else res[0]
    kv_bytes = float(np.sum(lens)) * cfg.kv_bytes_per_token()
    step_bytes = cfg.streamed_params() * 2 + kv_bytes
    line = {"metric": METRIC, "value": main["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": main["steps"],
            "warmup": W, "ms_per_step": main["ms_per_step"], "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, "batch": B, "gamma": GAMMA, "k": k if name != "verify_plain_decode" else 0,
                       "context": int(n0), "algorithmic_gb_per_step": step_bytes / 1e9,
                       "achieved_gbs": step_bytes / (main["ms_per_step"] * 1e-3) / 1e9, **{f"k{kk}": v for kk, v in res.items()}}}
    if 0 in res and k in res and name != "verify_plain_decode":
        line["config"]["speedup_vs_plain_decode"] = res[k]["tokens_per_s"] / res[0]["tokens_per_s"]
    if name == "k_sweep_long_context_b1":
        # the headline of this line is the best window; every k is in config
        best = max(res, key=lambda kk: res[kk]["tokens_per_s"])
        line["value"], line["ms_per_step"], line["steps"] = res[best]["tokens_per_s"], res[best]["ms_per_step"], res[best]["steps"]
        line["config"]["k"] = best
        line["config"]["speedup_by_k"] = {str(kk): res[kk]["tokens_per_s"] / res[0]["tokens_per_s"] for kk in res}
    print(json.dumps(line), flush=True)
    ctx.close()
    return 0


def run_drafted(args, cs, inputs, dev):
    """CopySpec merged with a draft model (Sec. 3.3) at the 8B shape: a 1B-class draft model
    (16 layers, d 2048, 32/8 heads of 64, FFN 8192, same vocabulary) proposes delta tokens where
    the search finds no match.  Scripted target: the stream alternates spans lifted from the
    4,096-token context with stretches that follow the draft model's own greedy choice three
    times out of four (built with the draft model on the GPU before the timed runs), so that both
    kinds of draft are partly accepted.  One line: the merged loop at delta = 3, with delta = 5,
    copy only (delta = 0, same host-driven loop) and plain decoding beside it."""
    import torch
    cfg = inputs.LLAMA8B
    dcfg = inputs.ModelConfig(n_layers=16, d_model=2048, n_heads=32, n_kv_heads=8, head_dim=64, d_ffn=8192,
                              vocab=cfg.vocab, rope_theta=500000.0, rms_eps=1e-5)
    n0, max_new, k = 4096, 768, K_DRAFT
    stride, max_seq = n0 + max_new + 64, n0 + max_new + k + 64
    tctx = cs.Context(cfg, inputs.make_weights(cfg, seed=0, device=str(dev)), max_seq=max_seq, max_batch=1, k_max=k)
    dctx = cs.Context(dcfg, inputs.make_weights(dcfg, seed=1, device=str(dev)), max_seq=max_seq, max_batch=1, k_max=15)
    g = torch.Generator(device=dev); g.manual_seed(1)
    kv_t, kv_d = tctx.alloc_kv(), dctx.alloc_kv()
    for kv, c in ((kv_t, cfg), (kv_d, dcfg)):
        for layer in range(c.n_layers):
            kv[layer, :, :, :, :n0 - 1, :] = torch.randn(2, 1, c.n_kv_heads, n0 - 1, c.head_dim, device=dev,
                                                          generator=g).to(torch.bfloat16)
    rng = np.random.default_rng(0)
    context = inputs.zipf_tokens(rng, n0, cfg.vocab, 1.1).astype(np.int32)
    # ---- the script, built with the draft model itself (single-row greedy steps)
    kvl = torch.tensor([n0 - 1], dtype=torch.int32, device=dev)
    last = torch.tensor([int(context[-1])], dtype=torch.int32, device=dev)
    zero = torch.zeros(1, dtype=torch.int32, device=dev)
    script = []
    while len(script) < max_new:
        if rng.random() < 0.5:
            src = int(rng.integers(0, n0 - 64))
            span, follow = [int(t) for t in context[src:src + int(rng.integers(20, 60))]], False
        else:
            span, follow = [None] * int(rng.integers(10, 30)), True
        for t in span:
            _, ot, _ = dctx.cs_verify_step(last, None, zero, kv_d, kvl)      # caches `last`, predicts the next token
            if follow:
                t = int(ot[0, 0]) if rng.random() < 0.75 else int(inputs.zipf_tokens(rng, 1, cfg.vocab, 1.1)[0])
            script.append(t)
            last.fill_(t)
    script = np.asarray(script[:max_new], dtype=np.int32)
    script_d = torch.from_numpy(script).to(dev)
    h = np.zeros((1, stride), dtype=np.int32)
    h[0, :n0] = context
    res = {}
    for label, kk, delta in (("copy_and_draft_d3", k, 3), ("copy_and_draft_d5", k, 5), ("copy_only", k, 0), ("plain_decode", 0, 0)):
        hd = torch.from_numpy(h).to(dev)
        ld = torch.tensor([n0], dtype=torch.int32, device=dev)
        kvl_t = torch.tensor([n0 - 1], dtype=torch.int32, device=dev)
        kvl_d = torch.tensor([n0 - 1], dtype=torch.int32, device=dev)
        new = max_new if kk else min(max_new, 4 * args.steps)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        st = tctx.cs_decode_loop_drafted(dctx if delta else None, hd, ld, kv_t, kvl_t, kv_d if delta else None,
                                         kvl_d if delta else None, GAMMA, kk, delta, new, script=script_d)
        torch.cuda.synchronize()
        sec = time.perf_counter() - t0
        if hd[0, n0:n0 + new].cpu().tolist() != script[:new].tolist():
            raise RuntimeError("the loop did not reproduce the script")
        res[label] = {"tokens_per_s": st["emitted"] / sec, "ms_per_step": sec / st["steps"] * 1e3, "steps": st["steps"],
                      "copy_attempts": st["attempts"], "mean_tau_copy": st["accepted"] / max(1, st["attempts"]),
                      "draft_attempts": st["draft_attempts"],
                      "mean_tau_draft": st["draft_accepted"] / max(1, st["draft_attempts"])}
    main_r = res["copy_and_draft_d3"]
    line = {"metric": METRIC, "value": main_r["tokens_per_s"], "unit": UNIT, "n_gpus": 1, "steps": main_r["steps"],
            "warmup": 0, "ms_per_step": main_r["ms_per_step"], "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "drafted_b1_k10", "batch": 1, "gamma": GAMMA, "k": k, "delta": 3, "context": n0,
                       "draft_model": "16L d2048 H32/8 Dh64 F8192 V128256", "timing": "host wall clock around the whole loop "
                       "(it synchronises every step)", **res,
                       "speedup_vs_plain_decode": {lab: r["tokens_per_s"] / res["plain_decode"]["tokens_per_s"] for lab, r in res.items()}}}
    print(json.dumps(line), flush=True)
    tctx.close(); dctx.close()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="verify",
                    choices=["verify", "verify_plain_decode", "long_context_b1_k10", "long_context_b8_k20", "k_sweep_long_context_b1", "prefill_b1_4096",
                             "multi_turn_b16_k10", "match_search", "drafted_b1_k10"],
                    help="verify = the benchmark; the others are additional single-GPU measurements")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: keep only this many of the 32 layers (small case for ncu captures; "
                         "not the benchmark workload)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)
    if args.workload != "verify":
        return run_workload(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
