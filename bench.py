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
per step) over W warm-up and exactly K timed steps with everything resident in HBM; the
same K steps are then repeated as further groups (`repeats`: median, p10, p90).  `e2e`
drives the same W + K steps from pinned host buffers through cs_step_host (one C call per
step: copies in, search, verify, copies out, host append), all inside the timed region.
`roofline` comes from a timeline of the same step taken inside the running pipeline
(cs_set_stamps).  `config` also carries the other two parts of the metric: plain one-token
decoding from the same kernels (k = 0, same cache) and the match search alone on the
64 x 32,768-token workload, with the CPU oracle's scan and dictionary beside it.
With N > 1 every rank runs an independent replica (the path does not shard).
`--impl reference` times the CPU oracle, as it stands, on a bounded sample.
"""
from __future__ import annotations

import argparse
import hashlib
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
SAMPLE_LAYERS = 4          # decoder layers of the CPU oracle's bounded sample

# DRAM counters of the dominant kernel, written beside its ncu summary: `key = value` lines
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "k_gemm_tc_verify8b_2layer_ncu_traffic.txt")
KERNEL_SOURCES = [os.path.join(ROOT, "paper_2502_08923_b200", "csrc", f) for f in ("cs_gemm.cu", "cs_common.cuh")]


def _kernel_hash():
    h = hashlib.sha256()
    for path in KERNEL_SOURCES:
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def _ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from the
    committed capture, or None when there is none or the kernel's source changed since."""
    try:
        kv = {}
        for line in open(TRAFFIC_FILE):
            if "=" in line and not line.lstrip().startswith("#"):
                k, v = line.split("=", 1)
                kv[k.strip()] = v.strip()
        if kv.get("kernel_source_sha256_16") != _kernel_hash():
            return None
        return float(kv["dram_bytes_per_projection_launch"])
    except Exception:
        return None


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
                                          "-lms", "50", "-i", str(self.index)],
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


def _case(n_steps, vocab):
    """History and script of the workload for n_steps steps (the context grows past 4,096 tokens
    only when more steps are asked for than its token paths have room for)."""
    from paper_2502_08923_b200 import inputs
    taus = _taus(n_steps)
    ctx_len = KV_START
    while True:
        try:
            hist, script = inputs.tau_controlled_case(np.random.default_rng(0), taus, GAMMA, K_DRAFT, ctx_len, vocab)
            return taus, hist, script
        except ValueError:
            ctx_len += 1024


# --------------------------------------------------------------------- CPU oracle leg
def oracle_sample(weights_cpu, kv_first_layers, hist, script, taus, n_steps, warmup):
    """Times the oracle, as it stands and through its public calls only, on a bounded sample of
    the workload: the scripted generation loop (search, gather, verification forward, acceptance,
    append) of a SAMPLE_LAYERS-layer slice of the 8B-class model with the full embedding and
    LM head, warm-up steps first, then n_steps timed steps.  The measured time per step of that
    slice is what `ms_per_step` reports; the whole model's step is extrapolated from it and a
    zero-layer forward (embedding, final norm, LM head) as head + 32 * (slice - head) / layers.
    Returns a dict with tokens/s (extrapolated) and the details."""
    from oracle import copyspec_oracle as O
    from paper_2502_08923_b200 import inputs
    import threadpoolctl
    cfg = inputs.LLAMA8B
    cfg_s, cfg_0 = inputs.sliced(cfg, SAMPLE_LAYERS), inputs.sliced(cfg, 0)
    n0 = len(hist)
    # embedding + final norm + LM head alone: one block through a model without layers
    head = O.Model(cfg_0, weights_cpu, contract=True, cache_weights=True)
    c0 = O.KVCache(cfg_0, 1, n0 + K_DRAFT + 1, dtype=np.float32)
    block = [int(hist[-1])] + [int(t) for t in script[:K_DRAFT]]
    head.forward_block(block, n0 - 1, c0, 0)
    ts = []
    for _ in range(3):
        t0 = time.perf_counter()
        head.forward_block(block, n0 - 1, c0, 0)
        ts.append(time.perf_counter() - t0)
    t_head = float(np.median(ts))
    del head
    # the scripted loop on the slice
    model = O.Model(cfg_s, weights_cpu, contract=True, cache_weights=True)
    tok_w, tok_t = sum(t + 1 for t in taus[:warmup]), sum(t + 1 for t in taus[warmup:warmup + n_steps])
    cache = O.KVCache(cfg_s, 1, n0 + tok_w + tok_t + K_DRAFT + 1, dtype=np.float32)
    cache.a[:, :, 0, :, :n0 - 1, :] = kv_first_layers
    h = [int(t) for t in hist]
    t0 = time.perf_counter()
    O.decode_loop(model, cache, 0, h, GAMMA, K_DRAFT, O.LATEST, tok_w, script=script[:tok_w])     # warm-up (converts the weights)
    t_warm = time.perf_counter() - t0
    trace = []
    t0 = time.perf_counter()
    O.decode_loop(model, cache, 0, h, GAMMA, K_DRAFT, O.LATEST, tok_t, script=script[tok_w:tok_w + tok_t], trace=trace)
    t_slice = (time.perf_counter() - t0) / max(1, len(trace))
    if len(trace) != n_steps or h[n0:] != [int(t) for t in script[:tok_w + tok_t]]:
        raise RuntimeError("the oracle's sample did not follow the script")
    t_full = t_head + cfg.n_layers * max(0.0, t_slice - t_head) / SAMPLE_LAYERS
    tokens_per_step = tok_t / n_steps
    cores = max([p.get("num_threads", 1) for p in threadpoolctl.threadpool_info()] + [1])
    return {"value": tokens_per_step / t_full, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": (f"{n_steps} timed steps (after {warmup} warm-up steps, {t_warm:.1f} s) of the scripted loop - search, gather, "
                       f"forward over an 11-row block and 4,096+ cached positions, acceptance, append - on a {SAMPLE_LAYERS}-layer slice "
                       f"of the 32-layer model with the full embedding and LM head: {t_slice * 1e3:.0f} ms per step measured; "
                       f"a zero-layer forward (embedding, final norm, LM head) takes {t_head * 1e3:.0f} ms; value = tokens per step / "
                       f"(head + 32 * (slice - head) / {SAMPLE_LAYERS}) = the whole model extrapolated"),
            "ms_per_step_sample": t_slice * 1e3, "ms_per_step_full_model_extrapolated": t_full * 1e3,
            "tokens_per_step": tokens_per_step}


def _oracle_inputs_cpu(cfg, n_ctx, seed=0):
    """The weights of the first SAMPLE_LAYERS layers, the embedding, the LM head and the K/V fill of
    those layers, drawn on the CPU with the bench's recipe (used when no GPU copy exists)."""
    import torch
    from paper_2502_08923_b200 import inputs
    w = inputs.make_weights(inputs.sliced(cfg, SAMPLE_LAYERS), seed=seed, device="cpu")
    kv = inputs.synthetic_kv(inputs.sliced(cfg, SAMPLE_LAYERS), 1, n_ctx, n_ctx, seed=1, device="cpu")
    return w, kv[:, :, 0].float().numpy()


def run_reference(args):
    rank, world, _ = _dist()
    if rank != 0:
        return 0
    from paper_2502_08923_b200 import inputs
    cfg = inputs.LLAMA8B
    steps = args.steps
    taus, hist, script = _case(args.warmup + steps, cfg.vocab)
    w, kv = _oracle_inputs_cpu(cfg, len(hist) - 1)
    res = oracle_sample(w, kv, hist, script, taus, steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": args.warmup, "ms_per_step": res["ms_per_step_sample"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "gamma": GAMMA, "k": K_DRAFT, "batch": 1, "kv_start": len(hist) - 1,
                       "ms_per_step_is": f"the measured step of the {SAMPLE_LAYERS}-layer sample; value is extrapolated to 32 layers",
                       "ms_per_step_full_model_extrapolated": res["ms_per_step_full_model_extrapolated"]},
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


def match_search_part(dev, n_timed=30):
    """Third part of the metric: the search alone on the 64 x 32,768-token workload (gamma 3, k 10):
    GPU time per sequence with the histories in L2 (warm) and after an L2 flush (cold), and the CPU
    oracle's scan and gamma-gram dictionary on the host cores (one thread, a sample of sequences)."""
    import torch
    from oracle import copyspec_oracle as O
    from paper_2502_08923_b200 import binding as cs, inputs
    hist, _, _ = inputs.match_search_histories()
    B, n = hist.shape
    hd = torch.from_numpy(hist).to(dev)
    ld = torch.full((B,), n, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    bufs = cs.cs_find_match(hd, ld, GAMMA, K_DRAFT)
    out = {"workload": f"{B} x {n} int32 histories, Zipf(1.1), 16 planted spans each; gamma {GAMMA}, k {K_DRAFT}"}
    for mode in ("warm", "cold"):
        ts = []
        for i in range(5 + n_timed):
            if mode == "cold":
                flush.fill_(i & 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cs.cs_find_match(hd, ld, GAMMA, K_DRAFT, out=bufs)
            e1.record()
            torch.cuda.synchronize()
            if i >= 5:
                ts.append(e0.elapsed_time(e1) * 1e3)
        out[f"gpu_{mode}_us_per_seq"] = float(np.median(ts)) / B
    out["gpu_cold_gbs"] = B * n * 4 / (out["gpu_cold_us_per_seq"] * B) / 1e3
    mp = bufs[0].cpu().numpy()
    sample = list(range(0, B, 8))
    t0 = time.perf_counter()
    got = [O.find_match(hist[b], n, GAMMA, O.LATEST) for b in sample]
    out["cpu_oracle_scan_us_per_seq"] = (time.perf_counter() - t0) / len(sample) * 1e6
    if got != [int(mp[b]) for b in sample]:
        raise RuntimeError("GPU search and oracle scan disagree")
    tb, tl = 0.0, 0.0
    for b in sample[:4]:
        d = O.GammaGramDict(GAMMA)
        t0 = time.perf_counter()
        d.extend(hist[b].tolist())
        tb += time.perf_counter() - t0
        t0 = time.perf_counter()
        for _ in range(100):
            p = d.lookup(O.LATEST)
        tl += (time.perf_counter() - t0) / 100
        if p != int(mp[b]):
            raise RuntimeError("GPU search and oracle dictionary disagree")
    out["cpu_oracle_dict_build_us_per_seq"] = tb / 4 * 1e6
    out["cpu_oracle_dict_lookup_us_per_seq"] = tl / 4 * 1e6
    out["cpu_threads"] = 1
    del flush
    return out


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
    W, K, G = args.warmup, args.steps, max(1, args.repeats)
    taus, hist, script = _case(W + K, cfg.vocab)
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
    hist0 = hist_d.clone()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reset_state():
        hist_d.copy_(hist0)
        len_d.fill_(n0)
        kvlen_d.fill_(n0 - 1)

    def run_group(k):
        """W warm-up steps, then exactly K timed steps of the device-resident loop from the
        workload's initial state.  Returns (ms of the K steps, tokens they emitted, launches per step)."""
        reset_state()
        ctx.cs_loop_begin(hist_d, len_d, kv, kvlen_d, GAMMA, k, max_new, script=script_d)
        launches = ctx.cs_loop_launches_per_step()
        ctx.cs_loop_steps(W)
        st0, _ = ctx.cs_loop_poll()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.cs_loop_steps(K)
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        st1, _ = ctx.cs_loop_poll()
        ctx.cs_loop_end()
        if st1["steps"] - st0["steps"] != K:
            raise RuntimeError(f"loop ran {st1['steps'] - st0['steps']} steps, expected {K}")
        return ms, st1["emitted"] - st0["emitted"], launches, st1

    # ---- the contract's number: group 0; the same W + K steps again as repeats ------------
    sampler = ClockSampler(local)
    sampler.start()
    groups = [run_group(K_DRAFT) for _ in range(G)]
    clocks = sampler.stop()
    ms, emitted, launches_per_step, st1 = groups[0]
    expect = sum(t + 1 for t in taus[W:W + K])
    if any(g[1] != expect for g in groups):
        raise RuntimeError(f"a group emitted {[g[1] for g in groups]} tokens, expected {expect}")
    ms, value = aggregate_replicas(ms, emitted, world, dev)
    per_step = sorted(g[0] / K for g in groups)
    repeats = {"groups": G, "steps_per_group": K, "ms_per_step_median": float(np.median(per_step)),
               "ms_per_step_p10": float(np.percentile(per_step, 10)), "ms_per_step_p90": float(np.percentile(per_step, 90)),
               "ms_per_step_all": [g[0] / K for g in groups]}

    # ---- plain one-token decoding from the same kernels, same cache (k = 0) ---------------
    plain = None
    if not args.no_extras:
        pms, pem, _, _ = run_group(0)
        plain = {"tokens_per_s": pem / (pms * 1e-3), "ms_per_step": pms / K, "steps": K}

    # ---- end to end from pinned host buffers: the same W + K steps, one cs_step_host call per
    # step (tokens the device lacks, length and script row host -> device, search + verify,
    # accepted length and tokens device -> host, the host appends)
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
    ctx.cs_step_host_reset()

    def host_step(n, e, new_tokens):
        scr_p[0].copy_(script_pad[e:e + K_DRAFT + 1])
        ctx.cs_step_host(hist_p, len_p, hist_e, len_e, kv, kvlen_d, GAMMA, K_DRAFT, acc_p, out_p, script_host=scr_p)
        tau = int(acc_p[0])
        return n + tau + 1, e + tau + 1, new_tokens * 4 + 4 + scr_p.numel() * 4, tau + 1

    n, e, new = n0, 0, n0            # the first call uploads the whole history, later ones what was appended
    for _ in range(W):
        n, e, _, new = host_step(n, e, new)
    barrier()
    t0 = time.perf_counter()
    e_start, h2d_total = e, 0
    for _ in range(K):
        n, e, nbytes, new = host_step(n, e, new)
        h2d_total += nbytes
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    if hist_p[0, n0:n].tolist() != script[:e].tolist() or e - e_start != expect:
        raise RuntimeError("host-driven steps did not reproduce the script")
    e2e_val = world * (e - e_start) / e2e_s

    # ---- timeline of the step inside the running pipeline -> roofline of the dominant kernel
    S = min(K, 24)
    stamps = torch.zeros(4096, dtype=torch.int64, device=dev)
    ctx.cs_set_stamps(stamps)
    reset_state()
    ctx.cs_loop_begin(hist_d, len_d, kv, kvlen_d, GAMMA, K_DRAFT, max_new, script=script_d)
    fams = ctx.cs_stamp_layout()
    nst = len(fams)
    rows = torch.zeros(S + 1, nst, dtype=torch.int64).pin_memory()
    ctx.cs_loop_steps(max(1, W - 1))
    for i in range(S + 1):
        ctx.cs_loop_steps(1)
        rows[i].copy_(stamps[:nst], non_blocking=True)      # stream-ordered: lands between two steps
    torch.cuda.synchronize()
    ctx.cs_loop_end()
    ctx.cs_set_stamps(None)
    ends = rows.numpy().astype(np.float64)
    fam_ms = {f: 0.0 for f in cs.STAMP_FAMILIES}
    fam_n = {f: 0 for f in cs.STAMP_FAMILIES}
    step_ms = []
    for i in range(1, S + 1):
        prev = ends[i - 1, nst - 1]
        step_ms.append((ends[i, nst - 1] - prev) * 1e-6)
        for j, f in enumerate(fams):
            fam_ms[f] += (ends[i, j] - (ends[i, j - 1] if j else prev)) * 1e-6 / S
            fam_n[f] += 1 if i == 1 else 0
    timeline_step = float(np.mean(step_ms))
    layer_bytes = cfg.n_layers * cfg.params_per_layer() * 2
    gemm_launches = max(1, fam_n["gemm"])
    peak, peak_kind = _peaks()
    achieved = layer_bytes / gemm_launches / (fam_ms["gemm"] / gemm_launches * 1e-3) / 1e9
    step_bytes = cfg.streamed_params() * 2 + (n0 - 1 + 0.5 * emitted) * cfg.kv_bytes_per_token()
    step_gbs = step_bytes / (ms / K * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "k_gemm_tc (layer projections)", "achieved": achieved, "peak": peak,
                "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind,
                "traffic": _ncu_traffic(),
                "bytes_per_launch": layer_bytes / gemm_launches, "launches_per_step": gemm_launches,
                "how": ("kernel time = end of its last CTA minus end of the preceding kernel's last CTA (%globaltimer stamps inside "
                        f"the pipelined step graph, mean of {S} consecutive steps); the families add up to the step"),
                "timeline_ms_per_step": fam_ms, "timeline_launches_per_step": fam_n, "timeline_step_ms": timeline_step,
                "dominant_kernel_share_of_step": fam_ms["gemm"] / timeline_step,
                "step": {"algorithmic_gb": step_bytes / 1e9, "achieved_gbs": step_gbs, "frac_of_measured_copy": step_gbs / peak,
                         "frac_of_8tbs": step_gbs / 8000.0}}

    line = None
    if rank == 0:
        search = None
        cpu = None
        if world == 1 and not args.no_extras:
            search = match_search_part(dev)
        if world == 1 and not args.no_cpu_baseline:
            # ---- CPU oracle on the host cores, bounded sample (rank 0, N = 1 only) ---------
            if cfg.n_layers >= SAMPLE_LAYERS:
                w_cpu = {"embed": weights["embed"].cpu(), "lm_head": weights["lm_head"].cpu(), "final_norm": weights["final_norm"].cpu(),
                         "layers": [{k2: v.cpu() for k2, v in weights["layers"][l].items()} for l in range(SAMPLE_LAYERS)]}
                kv_s = kv[:SAMPLE_LAYERS, :, 0, :, :n0 - 1, :].float().cpu().numpy()
                nc = min(K, 30)
                res = oracle_sample(w_cpu, kv_s, hist, script, taus, nc, 2)
                cpu = {k2: res[k2] for k2 in ("value", "unit", "cores", "kind", "sample")}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic",
                "config": {"workload": WORKLOAD, "model_shape": f"{cfg.n_layers}L d4096 H32/8 Dh128 F14336 V128256", "batch": 1,
                           "gamma": GAMMA, "k": K_DRAFT, "kv_start": n0 - 1, "kv_end": n0 - 1 + st1["emitted"],
                           "tokens_per_step": emitted / K, "l2": "inputs larger than L2 (15 GB of weights per step)",
                           "replicas": world, "draft_tokens_accepted_per_s": world * (emitted - K) / (ms * 1e-3),
                           "plain_decode_same_kernels": plain,
                           "speedup_vs_plain_decode": (value / world / plain["tokens_per_s"]) if plain else None,
                           "match_search": search},
                "repeats": repeats,
                "clocks": clocks,
                "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d_total // K, "d2h_bytes_per_step": d2h,
                        "steps": K, "ms_per_step": e2e_s / K * 1e3, "same_steps_as_value": True},
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
    cfg = inputs.LLAMA8B if args.layers <= 0 else inputs.sliced(inputs.LLAMA8B, args.layers)   # --layers: small case for ncu captures
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
    if name == "step_timeline":
        return run_step_timeline(args, cs, inputs, dev, cfg)
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


def run_step_timeline(args, cs, inputs, dev, cfg):
    """Per-kernel timeline of a loop step (cs_set_stamps: every launch leaves the time at which its last
    CTA finished; a kernel's share = its end minus its predecessor's end inside the replayed step
    graph, mean over --steps steps), for any batch, window and cache depth of the 8B shape (use
    --layers for a slice).  The script replays a span of the context, so every step accepts k tokens."""
    import torch
    B, k, S, W = args.batch, args.k, args.steps, args.warmup
    max_new = (W + S + 2) * (k + 1)
    n0 = args.kv + 1
    stride = (n0 + max_new + 67) // 4 * 4
    max_seq = n0 + max_new + k + 64
    weights = inputs.make_weights(cfg, seed=0, device=str(dev))
    ctx = cs.Context(cfg, weights, max_seq=max_seq, max_batch=B, k_max=k)
    kv = inputs.synthetic_kv(cfg, B, max_seq, n0 - 1, seed=1, device=str(dev))
    rng = np.random.default_rng(0)
    h = np.zeros((B, stride), dtype=np.int32)
    scripts = []
    for b in range(B):
        hh = rng.integers(0, cfg.vocab, size=n0).astype(np.int32)
        src = 100 + 37 * b
        hh[n0 - GAMMA:] = hh[src:src + GAMMA]
        h[b, :n0] = hh
        scripts.append(hh[src + GAMMA: src + GAMMA + max_new])
    hd = torch.from_numpy(h).to(dev)
    ld = torch.full((B,), n0, dtype=torch.int32, device=dev)
    kvl = torch.full((B,), n0 - 1, dtype=torch.int32, device=dev)
    stamps = torch.zeros(4096, dtype=torch.int64, device=dev)
    ctx.cs_set_stamps(stamps)
    ctx.cs_loop_begin(hd, ld, kv, kvl, GAMMA, k, max_new, script=torch.from_numpy(np.stack(scripts).astype(np.int32)).to(dev))
    fams = ctx.cs_stamp_layout()
    nst = len(fams)
    rows = torch.zeros(S + 1, nst, dtype=torch.int64).pin_memory()
    ctx.cs_loop_steps(W)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(S + 1):
        ctx.cs_loop_steps(1)
        rows[i].copy_(stamps[:nst], non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    st, _ = ctx.cs_loop_poll()
    ctx.cs_loop_end()
    ctx.close()
    ends = rows.numpy().astype(np.float64)
    iv = np.zeros(nst)
    for i in range(1, S + 1):
        for j in range(nst):
            iv[j] += (ends[i, j] - (ends[i, j - 1] if j else ends[i - 1, nst - 1])) / S / 1e3
    # launches of a step: search, set-up, embedding, then per layer QKV, attention, merge, O, gate/up, down, then LM head, acceptance, commit
    per_layer = (nst - 6) // cfg.n_layers
    if per_layer != 6:
        raise RuntimeError(f"unexpected launch layout: {nst} launches for {cfg.n_layers} layers")
    lay = iv[3:3 + 6 * cfg.n_layers].reshape(cfg.n_layers, 6)
    names = ["qkv", "attention", "merge", "o", "gate_up", "down"]
    line = {"metric": "step timeline", "value": float(iv.sum()), "unit": "us", "higher_is_better": False, "n_gpus": 1,
            "steps": S, "warmup": W, "ms_per_step": e0.elapsed_time(e1) / (S + 1), "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "step_timeline", "batch": B, "k": k, "kv": args.kv, "layers": cfg.n_layers,
                       "layer_us": float(lay.sum(1).mean()),
                       "per_layer_us": {n: float(lay[:, i].mean()) for i, n in enumerate(names)},
                       "search_us": float(iv[0]), "setup_us": float(iv[1]), "embed_us": float(iv[2]),
                       "lm_head_us": float(iv[-3]), "accept_us": float(iv[-2]), "commit_us": float(iv[-1]),
                       "emitted_per_step": st["emitted"] / max(1, st["steps"])}}
    print(json.dumps(line), flush=True)
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
    ap.add_argument("--repeats", type=int, default=5, help="groups of W + K steps (the first one is the reported value)")
    ap.add_argument("--no-extras", action="store_true",
                    help="profiling aid: leave out plain decoding and the match-search part (fewer launches under ncu)")
    ap.add_argument("--workload", default="verify",
                    choices=["verify", "verify_plain_decode", "long_context_b1_k10", "long_context_b8_k20", "k_sweep_long_context_b1", "prefill_b1_4096",
                             "multi_turn_b16_k10", "match_search", "drafted_b1_k10", "step_timeline"],
                    help="verify = the benchmark; the others are additional single-GPU measurements")
    ap.add_argument("--batch", type=int, default=1, help="step_timeline: sequences")
    ap.add_argument("--k", type=int, default=K_DRAFT, help="step_timeline: copied tokens per step")
    ap.add_argument("--kv", type=int, default=KV_START, help="step_timeline: cached tokens per sequence")
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
