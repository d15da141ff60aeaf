#!/usr/bin/env python
"""Benchmark of the mixed-batch step: tokens/s (decode + embedding rows) and roofline fraction.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3-7b|cfg2-1b|cfg4-7b-f<frac>]
  python bench.py --impl reference ...     # the CPU oracle on the host cores, same metric

A step is one hb_mixed_step over one synthetic mixed batch.  `value` times K steps with CUDA
events around the library calls (weights, KV pages and pool state resident in HBM; each call
copies its own small descriptor).  `e2e` repeats the K steps building the descriptor on the host
and reading logits and embeddings back to pinned host memory inside the timed region.
N > 1 runs N independent replicas (the method scales by replication; no collective).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mixed-batch tokens/s (decode+embed) on 1 B200 and % of roofline"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per launch of the projection GEMM come from a profiler capture, not from this program:
# a small data file beside the capture's summary holds the bytes per projection and the hash of the
# kernel source at capture time.  When the kernel source has changed since, the figure is stale and
# the line says `traffic: null`.
GEMM_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "gemm_tcgen05_cfg3-7b_layers2.traffic.txt")
GEMM_SOURCE = os.path.join(ROOT, "paper_2609_25405_b200", "csrc", "gemm_tcgen05.cu")


def gemm_traffic(shape_name, tokens_per_step):
    """(mean DRAM bytes per GEMM launch, note) from the capture's data file, or (None, why)."""
    import hashlib
    try:
        d = json.load(open(GEMM_TRAFFIC_FILE))
        h = hashlib.sha256(open(GEMM_SOURCE, "rb").read()).hexdigest()
    except Exception as e:
        return None, f"no capture data ({type(e).__name__})"
    if d.get("source_sha256") != h:
        return None, "kernel source changed since the capture"
    if d.get("shape") != shape_name or int(d.get("tokens_per_step", -1)) != int(tokens_per_step):
        return None, "capture is of another shape or step size"
    per = d["dram_bytes_per_launch"]
    return float(np.mean([per[k] for k in ("qkv", "o", "gate_up", "down")])), d.get("capture", "")


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def get_spec(name, cap_decode=0):
    from paper_2609_25405_b200 import workloads
    if name in workloads.SPECS:
        return workloads.SPECS[name]
    if name.startswith("cfg4-7b-f"):
        return workloads.sweep_spec(float(name[len("cfg4-7b-f"):]), cap_decode=cap_decode)
    raise SystemExit(f"unknown workload {name}")


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(gpu_index)], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [r.strip().split(", ") for r in open(self.f.name).read().strip().splitlines() if r.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for nm, v in zip(names, r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(nm)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------
# CPU baseline: the oracle, as it stands, on a bounded sample
# ------------------------------------------------------------------------------------------

class _SampleWeights:
    """Random float32 weights of the workload's shape for TIMING the oracle: one layer's tensors
    are generated and served for every layer, and only the first 1024 vocabulary rows exist
    (the sample's token ids stay below 1024, no logits are asked for)."""

    def __init__(self, shape, seed=0):
        rng = np.random.default_rng(seed)
        s = shape
        g = lambda r, c: rng.standard_normal((r, c), dtype=np.float32) * np.float32(0.02)
        self._layer = dict(attn_norm=np.ones(s.d, np.float32), ffn_norm=np.ones(s.d, np.float32),
                           wq=g(s.Hq * s.Dh, s.d), wk=g(s.Hkv * s.Dh, s.d), wv=g(s.Hkv * s.Dh, s.d),
                           wo=g(s.d, s.Hq * s.Dh), wg=g(s.F, s.d), wu=g(s.F, s.d), wd=g(s.d, s.F))
        self.tok_emb = g(1024, s.d)
        self.final_norm = np.ones(s.d, np.float32)
        self.lm_head = self.tok_emb

    def layer(self, l):
        return self._layer


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_sample(spec, n_tokens, repeats=1):
    """Times oracle.embed on one embedding request of n_tokens (last-token or mean pooling as the
    workload says), fp32.  Returns (tokens/s, seconds per sample)."""
    from oracle import transformer as T
    from paper_2609_25405_b200 import synth, consts
    shape = synth.SHAPES[spec.shape]
    W = _SampleWeights(shape)
    toks = np.random.default_rng(1).integers(0, 1024, n_tokens)
    mode = "last" if spec.pool_mode == consts.POOL_LAST else "mean"
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        T.embed(shape, W, toks, mode, dtype=np.float32)
        times.append(time.perf_counter() - t0)
    return n_tokens / float(np.mean(times)), times


def sample_tokens(spec):
    return min(spec.chunk, 512 if spec.shape == "7b" else 1024)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    spec = get_spec(args.workload)
    n = sample_tokens(spec) // 2
    for _ in range(args.warmup):
        oracle_sample(spec, n)
    t0 = time.perf_counter()
    _, times = oracle_sample(spec, n, repeats=args.steps)
    total = time.perf_counter() - t0
    value = n * args.steps / sum(times)
    cores = blas_threads()
    sample = (f"oracle.transformer.embed (fp32 numpy) on one {n}-token embedding request of the {spec.shape} shape "
              f"per step; one layer's random weights reused for all layers (timing only)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": spec.name, "sample_tokens": n},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": total}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
# config 5: synthetic iterative-retrieval trace, virtual-clock replay (1B shape)
# ------------------------------------------------------------------------------------------

def trace_line(n_sessions):
    import torch
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import synth, trace
    from paper_2609_25405_b200.engine import Engine
    shape = synth.SHAPES["1b"]
    sessions = trace.make_trace(shape.V, seed=1005, n_sessions=n_sessions)
    budget, chunk = 4096, 256
    max_pos = 2048 + 128 + 8
    P = shape.page_size
    n_pages = n_sessions * ((max_pos + P - 1) // P) + 64
    weights = B.DeviceWeights.random_on_device(shape, seed=0)
    eng = Engine(shape, weights, n_pages=n_pages, n_slots=n_sessions + 8, max_tokens=budget,
                 max_segs=n_sessions + budget // 16 + 8, max_pos=max_pos)
    t0 = time.perf_counter()
    out = trace.replay(sessions, eng, budget, chunk)
    wall = time.perf_counter() - t0
    status = eng.ctx.status_poll()
    line = {"metric": METRIC, "value": out["rows"] / out["busy_s"], "unit": UNIT, "n_gpus": 1, "steps": out["steps"],
            "warmup": 0, "ms_per_step": 1e3 * out["busy_s"] / max(out["steps"], 1), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": "cfg5-trace-1b", "shape": shape.name, "sessions": n_sessions,
                       "arrival_rate_per_s": 20.0, "token_budget": budget, "chunk": chunk, "scheduler": "IBS",
                       "clock": "virtual: advances by measured GPU time per step, jumps over idle gaps"},
            "rows": out["rows"], "expected_rows": trace.trace_tokens(sessions),
            "busy_s": out["busy_s"], "virtual_clock_s": out["clock_s"],
            "tokens_per_s_over_clock": out["rows"] / out["clock_s"], "host_wall_s": wall,
            "sessions_done": out["sessions_done"], "device_status": status}
    eng.close()
    return line


def run_trace(args):
    print(json.dumps(trace_line(args.sessions)))


def run_phases(args):
    """Shifting request mix (10 % / 50 % / 90 % embedding requests) on one GPU through the IBS
    scheduler: per-phase service rate of the same engine, nothing repartitioned between phases."""
    import torch
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import synth, trace
    from paper_2609_25405_b200.engine import Engine
    shape = synth.SHAPES[args.workload.split("-")[1]]
    n_req = args.sessions
    phases = trace.make_phases(shape.V, n_requests=n_req)
    budget, chunk = 4096, 512
    max_pos = 128 + 512 + 8
    P = shape.page_size
    n_pages = n_req * ((max_pos + P - 1) // P) + 64
    weights = B.DeviceWeights.random_on_device(shape, seed=0)
    eng = Engine(shape, weights, n_pages=n_pages, n_slots=n_req + 8, max_tokens=budget,
                 max_segs=n_req + budget // 16 + 8, max_pos=max_pos)
    per_phase, rows, busy, steps = [], 0, 0.0, 0
    for frac, sessions in zip((0.1, 0.5, 0.9), phases):
        out = trace.replay(sessions, eng, budget, chunk)
        per_phase.append({"embed_request_frac": frac, "rows": out["rows"], "steps": out["steps"],
                          "busy_s": out["busy_s"], "tokens_per_s": out["rows"] / out["busy_s"],
                          "mean_rows_per_step": out["rows"] / max(out["steps"], 1),
                          "expected_rows": trace.trace_tokens(sessions)})
        rows += out["rows"]; busy += out["busy_s"]; steps += out["steps"]
    status = eng.ctx.status_poll()
    line = {"metric": METRIC, "value": rows / busy, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": 0,
            "ms_per_step": 1e3 * busy / max(steps, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape.name, "requests_per_phase": n_req,
                       "token_budget": budget, "chunk": chunk, "scheduler": "IBS",
                       "sizes": "embedding 128 tokens; generation 128-token prompt + 512 decode steps"},
            "phases": per_phase, "free_pages_after": eng.kv.free_count(), "n_pages": n_pages,
            "device_status": status}
    print(json.dumps(line))
    eng.close()


# ------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------

def measure_mixed(args, workload, steps, warmup, dist=None, rank=0, world=1, local=0, weights_cache=None,
                  kv_arena=None, decode_alias=0, cap_decode=0, with_e2e=True, with_classes=True, sample_clocks=True):
    """Times `steps` mixed steps of one workload after `warmup` untimed ones.  Returns a dict of the
    rank-aggregated figures (max time over ranks, summed tokens)."""
    import torch
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import replicas, synth, workloads
    from paper_2609_25405_b200.engine import build_batch

    spec = get_spec(workload, cap_decode)
    if world > 1:   # independent replicas: each rank draws its own batch stream
        spec = workloads.MixSpec(**{**spec.__dict__, "seed": replicas.rank_seed(spec.seed, rank)})
    shape = synth.SHAPES[spec.shape]
    if args.layers:
        shape = shape.with_layers(args.layers)
    n_steps_total = warmup + steps
    max_pos = spec.ctx_hi + n_steps_total + 8 if spec.n_decode else spec.emb_hi + 8
    max_pos = max(max_pos, spec.emb_hi + 8)
    cfg = B.model_cfg(shape, max_pos)
    P = shape.page_size
    n_unique = min(decode_alias, spec.n_decode) if decode_alias else spec.n_decode
    dec_pages = n_unique * ((spec.ctx_hi + P - 1) // P + 1) + spec.n_decode * ((n_steps_total + P - 1) // P + 2)
    emb_pages = 3 * spec.budget // P + 32 * ((spec.emb_hi + P - 1) // P)
    n_pages = dec_pages + emb_pages
    max_segs = spec.n_decode + spec.budget // 16 + 8
    max_page_ids = spec.n_decode * ((max_pos + P - 1) // P) + (spec.budget // 16 + 8) * ((spec.emb_hi + P - 1) // P + 1)

    key = (shape.name, args.lora_rank)
    if weights_cache is not None and key in weights_cache:
        weights, lora = weights_cache[key]
    else:
        weights = B.DeviceWeights.random_on_device(shape, seed=0)
        lora = B.DeviceLora.random_on_device(shape, args.lora_rank) if args.lora_rank else None
        if weights_cache is not None:
            weights_cache[key] = (weights, lora)
    kv = B.KvCache(cfg, n_pages, arena=kv_arena)
    if kv_arena is None:
        kvb = kv.arena.view(torch.float16)
        step_e = 1 << 28
        for i in range(0, kvb.numel(), step_e):          # synthetic cached K/V: N(0,1)
            kvb[i:i + step_e].normal_(0.0, 1.0)
    pool = B.Pool(cfg, 256)
    ctx = B.Context(cfg, spec.budget, max_segs, max_page_ids)
    wl = workloads.MixedWorkload(spec, kv, pool, max_pos, decode_alias=decode_alias, shape=shape)
    for _ in range(args.packer_warm):                # reach the packer's steady state (host only)
        _, commit = wl.next_step()
        commit(advance_decode=False)
    entries_all, batches, work = [], [], []
    for _ in range(n_steps_total):
        entries, commit = wl.next_step()
        entries = [dict(e, pages=list(e["pages"])) for e in entries]
        commit()
        entries_all.append(entries)
        batches.append(build_batch(entries, P)[0])
        work.append(workloads.step_work(shape, entries))
    out_logits = torch.zeros((max_segs, shape.V), dtype=torch.float32, device="cuda")
    out_emb = torch.zeros((max_segs, shape.d), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()

    def run(i):
        ctx.mixed_step(batches[i], weights, kv, pool, out_logits, out_emb, stream, lora=lora)

    for i in range(warmup):
        run(i)
    torch.cuda.synchronize()
    if ctx.status_poll() != 0:
        raise SystemExit("device status set during warm-up")
    timed = list(range(warmup, n_steps_total))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    sampler = ClockSampler(local) if (rank == 0 and sample_clocks) else None
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    launches = 0
    for i in timed:
        run(i)
        launches += ctx.last_launch_count()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None

    # ---- end to end: host packing + call + read-back of logits / embeddings ----
    e2e_s, h2d, d2h = float("nan"), 0, 0
    if with_e2e:
        h_logits = torch.empty((max_segs, shape.V), dtype=torch.float32).pin_memory()
        h_emb = torch.empty((max_segs, shape.d), dtype=torch.float32).pin_memory()
        barrier()
        t0 = time.perf_counter()
        for i in timed:
            b = build_batch(entries_all[i], P)[0]
            ctx.mixed_step(b, weights, kv, pool, out_logits, out_emb, stream, lora=lora)
            nl, ne = b.desc.n_logit_rows, b.desc.n_emb_rows
            if nl:
                h_logits[:nl].copy_(out_logits[:nl], non_blocking=True)
            if ne:
                h_emb[:ne].copy_(out_emb[:ne], non_blocking=True)
            torch.cuda.synchronize()
            h2d += b.host_bytes()
            d2h += nl * shape.V * 4 + ne * shape.d * 4
        barrier()
        e2e_s = time.perf_counter() - t0

    # ---- per-class kernel timing (events around every launch, same steps) ----
    prof = None
    if with_classes:
        ctx.profile_enable(True)
        for i in timed:
            run(i)
        torch.cuda.synchronize()
        prof = ctx.profile_read()
        ctx.profile_enable(False)
    status = ctx.status_poll()

    tokens = sum(work[i]["T"] for i in timed)
    ms, e2e_ms, tokens = replicas.aggregate(dist, "cuda", ms, e2e_s * 1e3, tokens)
    K = len(timed)
    w = {k: float(np.mean([work[i][k] for i in timed])) for k in work[0]}
    ctx.close(); kv.close(); pool.close()
    del out_logits, out_emb, kv, pool, ctx
    return dict(spec=spec, shape=shape, ms=ms, e2e_ms=e2e_ms, tokens=tokens, K=K, w=w, prof=prof, clocks=clocks,
                launches=launches, status=status, h2d=h2d, d2h=d2h, decode_alias=decode_alias)


def step_roofline(w, step_ms, peaks, peak_kind):
    """The benchmark spec's roofline of a step: the slower of GEMM flop at the bf16 tensor peak and
    weight + KV bytes at the HBM rate, against the measured step time."""
    bytes_step = w["weight_bytes"] + w["kv_read_bytes"] + w["kv_write_bytes"]
    t_gemm_burst = w["gemm_flops"] / (peaks["bf16_tflops"] * 1e12)
    t_gemm_sust = w["gemm_flops"] / (peaks["bf16_tflops_sustained"] * 1e12)
    t_mem = bytes_step / (peaks["hbm_gbs"] * 1e9)
    return {"gemm_tflop": w["gemm_flops"] / 1e12, "attn_tflop": w["attn_flops"] / 1e12,
            "bytes_gb": bytes_step / 1e9, "t_gemm_ms_burst": t_gemm_burst * 1e3,
            "t_gemm_ms_sustained": t_gemm_sust * 1e3, "t_mem_ms": t_mem * 1e3,
            "bound": "tensor" if t_gemm_burst > t_mem else "hbm",
            "frac_of_burst_roof": max(t_gemm_burst, t_mem) * 1e3 / step_ms,
            "frac_of_sustained_roof": max(t_gemm_sust, t_mem) * 1e3 / step_ms,
            # nominal dense bf16 rate and HBM3e bandwidth of the part, for context only
            "frac_of_datasheet_roof": max(w["gemm_flops"] / 2250e12, bytes_step / 8.0e12) * 1e3 / step_ms,
            "peak_kind": peak_kind}


def short_entry(m, peaks, peak_kind, note=None):
    """One other configuration in brief: step time, tokens/s, its step roofline."""
    step_ms = m["ms"] / m["K"]
    r = step_roofline(m["w"], step_ms, peaks, peak_kind)
    e = {"workload": m["spec"].name, "steps": m["K"], "ms_per_step": step_ms, "value": m["tokens"] / (m["ms"] * 1e-3),
         "unit": UNIT, "tokens_per_step": m["w"]["T"], "decode_rows": m["spec"].n_decode,
         "decode_alias": m["decode_alias"], "bound": r["bound"], "roof_ms": max(r["t_gemm_ms_burst"], r["t_mem_ms"]),
         "frac_of_burst_roof": r["frac_of_burst_roof"], "device_status": m["status"]}
    if m["prof"]:
        e["kernel_classes_ms"] = {k: v[0] / m["K"] for k, v in m["prof"].items() if v[1]}
    if note:
        e["note"] = note
    return e


def other_configs(args, peaks, peak_kind, weights_cache):
    """The other benchmark configurations in brief (the 1B step, the five mixes of the 7B sweep, the
    retrieval trace), so that one default run shows all of them.  A configuration that fails reports
    its error here and leaves the headline alone."""
    import torch
    out = []

    def attempt(name, fn):
        try:
            out.append(fn())
        except BaseException as e:   # noqa: BLE001  (reported, never fatal to the headline)
            if isinstance(e, KeyboardInterrupt):
                raise
            out.append({"workload": name, "error": f"{type(e).__name__}: {e}"[:300]})
        torch.cuda.empty_cache()

    # the sweep reuses the 7B weights of the headline and ONE KV arena for its five mixes
    from paper_2609_25405_b200 import binding as B
    from paper_2609_25405_b200 import synth
    alias = 256
    fracs = (0.0, 0.25, 0.5, 0.75, 0.95)
    arena = None
    try:
        shape7 = synth.SHAPES["7b"]
        P = shape7.page_size
        n_total = 3 + 4
        worst = alias * ((2048 + P - 1) // P + 1) + 4096 * ((n_total + P - 1) // P + 2) + 3 * 4096 // P + 32 * (2048 // P) + 64
        nbytes = B.kv_arena_bytes(B.model_cfg(shape7, 4096), worst)
        arena = torch.empty(nbytes // 2, dtype=torch.int16, device="cuda")
        kvb = arena.view(torch.float16)
        for i in range(0, kvb.numel(), 1 << 28):
            kvb[i:i + (1 << 28)].normal_(0.0, 1.0)
    except BaseException as e:   # noqa: BLE001
        out.append({"workload": "cfg4-7b", "error": f"{type(e).__name__}: {e}"[:300]})
    if arena is not None:
        for f in fracs:
            name = f"cfg4-7b-f{f:g}"
            attempt(name, lambda: short_entry(
                measure_mixed(args, name, 4, 3, weights_cache=weights_cache, kv_arena=arena, decode_alias=alias,
                              with_e2e=False, with_classes=True, sample_clocks=False), peaks, peak_kind,
                note=f"decode rows read {alias} distinct cached contexts (the unaliased KV of 4096 rows at "
                     "context 2048 would be 1.1 TB); each row appends to a private tail page"))
        del arena, kvb
        torch.cuda.empty_cache()
    weights_cache.clear()
    torch.cuda.empty_cache()
    attempt("cfg2-1b", lambda: short_entry(
        measure_mixed(args, "cfg2-1b", 20, 5, weights_cache=weights_cache, with_e2e=False, sample_clocks=False),
        peaks, peak_kind))
    weights_cache.clear()
    torch.cuda.empty_cache()

    def trace_entry():
        t = trace_line(args.sessions)
        return {"workload": "cfg5-trace-1b", "value": t["value"], "unit": UNIT, "steps": t["steps"],
                "ms_per_step": t["ms_per_step"], "rows": t["rows"], "expected_rows": t["expected_rows"],
                "busy_s": t["busy_s"], "sessions_done": t["sessions_done"], "device_status": t["device_status"],
                "config": t["config"]}
    attempt("cfg5-trace-1b", trace_entry)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3-7b")
    ap.add_argument("--packer-warm", type=int, default=50, help="host-only packer steps before the first GPU step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the brief runs of the other configurations (1B step, 7B sweep, trace)")
    ap.add_argument("--decode-alias", type=int, default=0)
    ap.add_argument("--cap-decode", type=int, default=0,
                    help="sweep workloads: cap the decode rows at what fits in HBM unaliased (the step gets smaller)")
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (profiling on a small case)")
    ap.add_argument("--sessions", type=int, default=256, help="sessions of the cfg5-trace-1b workload")
    ap.add_argument("--gemm-walk", default="", help="tuning: force the projection GEMM's tile walk, 'band,hints' (see hb_gemm_set_walk)")
    ap.add_argument("--gemm-ctas", type=int, default=0, help="tuning: cap the CTAs of every projection GEMM launch")
    ap.add_argument("--lora-rank", type=int, default=0,
                    help="rank of a random low-rank adapter applied to the embedding rows (0 = none, the headline)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
        return

    # `--gpus N` started plainly (no launcher in the environment): start the N replica ranks here
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        from paper_2609_25405_b200 import replicas
        rcs = replicas.spawn_ranks([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)
        sys.exit(max(abs(r) for r in rcs))

    import torch

    if args.gemm_walk:
        from paper_2609_25405_b200 import binding as _B
        _B.gemm_set_walk(*[int(v) for v in args.gemm_walk.split(",")])
    if args.gemm_ctas:
        from paper_2609_25405_b200 import binding as _B
        _B.gemm_set_cta_limit(args.gemm_ctas)
    if args.workload.startswith("cfg5-trace"):
        run_trace(args)
        return
    if args.workload.startswith("phases-"):
        run_phases(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    weights_cache = {}
    m = measure_mixed(args, args.workload, args.steps, args.warmup, dist=dist, rank=rank, world=world, local=local,
                      weights_cache=weights_cache, decode_alias=args.decode_alias, cap_decode=args.cap_decode)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    spec, shape, w, prof, K = m["spec"], m["shape"], m["w"], m["prof"], m["K"]
    peaks, peak_kind = load_peaks()
    step_ms = m["ms"] / K
    step_roof = step_roofline(w, step_ms, peaks, peak_kind)
    # dominant kernel: the projection GEMM, launches timed one by one in the per-class pass
    gemm_ms, gemm_n = prof["gemm"]
    gemm_flops_launch = (w["gemm_flops"] - 2.0 * shape.d * shape.V * w["n_logit"]) * K / max(gemm_n, 1)
    ach_tf = gemm_flops_launch / (gemm_ms / max(gemm_n, 1) * 1e-3) / 1e12 if gemm_ms > 0 else None
    traffic, traffic_note = (None, "reduced layer count") if args.layers else gemm_traffic(spec.shape, w["T"])
    gemm_kernel = {"kernel": "hb_gemm_tcgen05_kernel (QKV, O, gate/up, down projections)", "bound": "tensor",
                   "achieved": ach_tf, "unit": "TFLOP/s", "peak": peaks["bf16_tflops_sustained"],
                   "frac": (ach_tf / peaks["bf16_tflops_sustained"]) if ach_tf else None,
                   "peak_kind": f"{peak_kind} cuBLAS bf16, sustained (launches timed one by one inside a long run, "
                                "no overlap between them); fp16 operands have the same nominal tensor rate as bf16",
                   "frac_of_burst": (ach_tf / peaks["bf16_tflops"]) if ach_tf else None,
                   "launches": gemm_n, "flops_per_launch": gemm_flops_launch,
                   "traffic": traffic, "traffic_from": traffic_note}
    # the two attention item lists, each timed alone in the per-class pass (in the step they share one launch)
    attention_kernels = {}
    dec_ms, dec_n = prof.get("attention", (0.0, 0))
    if dec_n and dec_ms > 0:
        gbs = w["kv_read_bytes_decode"] * K / (dec_ms * 1e-3) / 1e9
        attention_kernels["decode_items"] = {
            "kernel": "attn_varlen_kernel, decode splits alone (mma.sync body over paged KV)",
            "bound": "hbm", "achieved": gbs, "unit": "GB/s", "peak": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
            "bytes_per_launch": w["kv_read_bytes_decode"] * K / dec_n, "launches": dec_n,
            "note": "algorithmic bytes: keys and values the decode rows read; events around every launch, "
                    "~10 us of gap per launch included"}
    tc_ms, tc_n = prof.get("attention_tc", (0.0, 0))
    if tc_n and tc_ms > 0:
        tf = w["attn_flops_chunk"] * K / (tc_ms * 1e-3) / 1e12
        attention_kernels["chunk_tiles"] = {
            "kernel": "attn_varlen_kernel, chunk tiles alone (tcgen05 body)", "bound": "tensor", "achieved": tf,
            "unit": "TFLOP/s", "peak": peaks["bf16_tflops"], "frac": tf / peaks["bf16_tflops"],
            "flops_per_launch": w["attn_flops_chunk"] * K / tc_n, "launches": tc_n,
            "note": "4 Dh flop per visible (query, key, head) triple, chunk rows of all lengths; against the burst peak"}
    # The headline fraction is the STEP's: the whole mixed step against the slower of its GEMM flop at
    # the measured bf16 burst peak and its weight + KV bytes at the measured HBM rate.
    if step_roof["bound"] == "tensor":
        ach, peak, unit = w["gemm_flops"] / (step_ms * 1e-3) / 1e12, peaks["bf16_tflops"], "TFLOP/s"
    else:
        ach, peak, unit = step_roof["bytes_gb"] / (step_ms * 1e-3), peaks["hbm_gbs"], "GB/s"
    roofline = {"scope": "step", "bound": step_roof["bound"], "achieved": ach, "peak": peak, "unit": unit,
                "frac": ach / peak, "traffic": traffic,
                "peak_kind": f"{peak_kind}: cuBLAS bf16 burst / copy bandwidth (the conservative denominators; "
                             f"against the sustained cuBLAS rate the step is at {step_roof['frac_of_sustained_roof']:.3f})",
                "traffic_scope": "mean DRAM bytes per projection-GEMM launch (profiler capture), see gemm_kernel",
                "gemm_kernel": gemm_kernel, "attention_kernels": attention_kernels}
    breakdown = {k: {"ms_per_step": v[0] / K, "launches_per_step": v[1] / K} for k, v in prof.items()}
    line = {"metric": METRIC, "value": m["tokens"] / (m["ms"] * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f16", "data": "synthetic",
            "precision": "bf16 random-init weights, repacked once to fp16; fp16 x fp16 operands (weights, "
                         "activations, KV cache) on the tensor cores with fp32 accumulation; fp32 residual "
                         "stream, norms, softmax and pooling",
            "config": {"workload": spec.name, "shape": shape.name, "tokens_per_step": w["T"],
                       "decode_rows": spec.n_decode, "chunk": spec.chunk, "token_budget": spec.budget,
                       "l2": "inputs larger than L2 (weights and KV pages are re-streamed every step)",
                       "replicas": world, "decode_alias": args.decode_alias, "lora_rank": args.lora_rank},
            "clocks": m["clocks"], "e2e": {"value": m["tokens"] / (m["e2e_ms"] * 1e-3), "unit": UNIT,
                                           "h2d_bytes_per_step": m["h2d"] / K, "d2h_bytes_per_step": m["d2h"] / K},
            "gpu_launches": m["launches"], "roofline": roofline, "step_roofline": step_roof,
            "kernel_classes": breakdown, "device_status": m["status"]}
    if dist is not None:
        dist.destroy_process_group()
    if world == 1 and not args.no_other_configs and args.workload == "cfg3-7b" and not args.layers \
            and not args.lora_rank:
        line["other_configs"] = other_configs(args, peaks, peak_kind, weights_cache)
    if not args.no_cpu_baseline:
        n = sample_tokens(spec)
        v, times = oracle_sample(spec, n)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                "sample": f"oracle.transformer.embed (fp32 numpy) on one {n}-token embedding request "
                                          f"of the {spec.shape} shape, {times[0]:.1f} s; one layer's random weights "
                                          f"reused for all layers (timing only)"}
    print(json.dumps(line))


if __name__ == "__main__":
    main()
