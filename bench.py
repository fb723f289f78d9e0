#!/usr/bin/env python
"""Benchmark of the speculative-sampling verification path on B200.

A "step" is one speculative iteration over one batch: K draft steps, one target verification
pass over K+1 rows per sequence, accept/reject/resample and cache bookkeeping.  The headline
value is generated tokens per second (speculative); the same run also times plain
autoregressive decoding, the verification pass alone (batch of the workload, and batch 1 at a
2048-token context with 1, 4 and 5 rows), and attributes device time to the kernel that streams
the weights for the roofline figure.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With --gpus N > 1 and no launcher in the environment the script re-executes itself under
torch.distributed.run, one replica per GPU.  Prints ONE JSON line (rank 0).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "generated tok/s, speculative vs autoregressive; verify-step HBM GB/s vs peak"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0     # sustained cuBLAS bf16 on this pool when the measured file is absent
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes (read + write) of one verify launch of the forward kernel, from the profiler captures
# summarised under profiles/.  A capture of the full 32-layer 7B pass would hold the whole model under
# the profiler, so the 7B workloads are scaled from a four-layer cut of the same kernel: the layers are
# identical and the LM head is the same, hence
#     traffic(32 layers) = head + 8 * (traffic(4 layers) - head),   head = LM-head matrix + logits rows.
# An entry is dropped (None) when the kernel has changed since its capture.
NCU_TRAFFIC = {
    # workload: (captured workload, dram bytes of the captured launch, layers captured)
    "llama-7b-b8": ("llama-7b-l4-b8", 3.1158e9, 4),        # profiles/forward_kernel_llama-7b-l4-b8_verify.md
    "llama-7b-l4-b8": ("llama-7b-l4-b8", 3.1158e9, 4),
    "llama-7b-l4-ctx8k": ("llama-7b-l4-ctx8k", 2.4807e9, 4),  # profiles/forward_kernel_llama-7b-l4-ctx8k_verify.md
    "neox-1.4b": ("neox-1.4b", 2.6746e9, 24),               # profiles/forward_kernel_neox-1.4b_verify.md
}

# bench workloads: name -> preset (+ overrides)
WORKLOADS = {
    "llama-7b-b8": dict(preset="llama-7b"),
    "llama-7b-b1": dict(preset="llama-7b", batch=1, prompt=2048),
    "neox-1.4b": dict(preset="neox-1.4b"),
    "neox-2.7b": dict(preset="neox-2.7b"),
    "neox-12b": dict(preset="neox-12b"),
    # four-layer cuts of the 7B shape, small enough for a full profiler capture: the same per-layer phases;
    # time and bytes scale with the layers
    "llama-7b-l4-ctx8k": dict(preset="llama-7b", batch=1, prompt=8192, layers=4),
    "llama-7b-l4-b8": dict(preset="llama-7b", layers=4),
    "tiny": dict(preset="tiny"),
}
DEFAULT_WORKLOAD = "llama-7b-b8"


def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------ bytes the method must move
def weight_bytes(arch) -> int:
    """Bytes of matrices streamed by one forward (all layers + LM head), model dtype."""
    es = 2 if arch.dtype else 4
    d, F = arch.d_model, arch.d_ff
    per_layer = 3 * d * d + d * d + arch.d_in * d + d * F
    return (arch.n_layers * per_layer + arch.vocab * d) * es


def verify_step_bytes(arch, batch, K, ctx_lens) -> int:
    """Algorithmic bytes of one verification pass: weights once, embedding rows, KV read of
    every sequence's context plus the new rows, KV write, draft rows q and the uniforms."""
    es = 2 if arch.dtype else 4
    M = K + 1
    kv_tok = 2 * arch.n_layers * arch.d_model * es
    b = weight_bytes(arch) + batch * M * arch.d_model * es
    b += sum((int(n) + M) * kv_tok for n in ctx_lens) + batch * M * kv_tok
    b += batch * K * arch.vocab * 4 + batch * M * 4
    return b


def scaled_traffic(workload, arch, rows):
    """DRAM traffic of one verify launch for `workload`, from the capture table (None if not captured)."""
    ent = NCU_TRAFFIC.get(workload)
    if ent is None:
        return None
    _, dram, layers = ent
    if layers == arch.n_layers:
        return float(dram)
    head = arch.vocab * arch.d_model * (2 if arch.dtype else 4) + rows * arch.vocab * 4
    return float(head + (arch.n_layers / layers) * (dram - head))


# ------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------ model construction
def random_weights_on_device(arch, seed, torch, late_scale=1.0, late_from=0):
    """Random-init tensors drawn on the device (N(0, 0.02); gains 1 + N(0, 0.02)), ABI order."""
    from paper_2311_04951_b200 import synth
    g = torch.Generator(device="cuda")
    out = []
    for i, name in enumerate(synth.tensor_names(arch)):
        shape = synth.tensor_shape(arch, name)
        if shape is None:
            out.append(None)
            continue
        g.manual_seed(seed * 100003 + i)
        t = torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * 0.02
        base = name.split(".")[-1]
        if base.endswith("_g"):
            t += 1.0
        if "." in name and base in ("w_o", "w_out", "b_o", "b_out") and int(name.split(".")[0][1:]) >= late_from:
            t *= late_scale
        out.append(t.to(torch.bfloat16) if (len(shape) == 2 and arch.dtype) else t)
    return out


def weights_to_host(tensors, torch):
    """Device tensors -> the numpy arrays the oracle takes (bf16 matrices as uint16 bit patterns): a copy
    of the inputs as data, no arithmetic."""
    out = []
    for t in tensors:
        if t is None:
            out.append(None)
        elif t.dtype == torch.bfloat16:
            out.append(t.view(torch.int16).cpu().numpy().view(np.uint16))
        else:
            out.append(t.cpu().numpy())
    return out


def resolve(workload):
    from paper_2311_04951_b200 import synth
    w = dict(WORKLOADS[workload])
    cfg = dict(synth.PRESETS[w.pop("preset")])
    layers = w.pop("layers", None)
    cfg.update(w)
    if layers:
        cfg["target"] = cfg["target"].replace(n_layers=layers)
    return cfg


def late_scaling(cfg):
    # layer-skip drafts need correlated exits: damp the late layers' output projections
    return dict(late_scale=0.2, late_from=4) if cfg["draft"] == "prefix:4" else {}


def expected_tokens_per_iteration(alpha, K):
    """Closed form for i.i.d. acceptance with per-token rate alpha: (1 - alpha^(K+1)) / (1 - alpha)."""
    if alpha >= 1.0:
        return float(K + 1)
    return (1.0 - alpha ** (K + 1)) / (1.0 - alpha)


def run_ours(args, rank, world):
    import torch
    from paper_2311_04951_b200 import binding as B, engine, synth

    local = int(os.environ.get("LOCAL_RANK", 0))
    if local >= torch.cuda.device_count():
        raise RuntimeError(f"rank {rank}: local rank {local} has no GPU ({torch.cuda.device_count()} visible)")
    torch.cuda.set_device(local)
    cfg = resolve(args.workload)
    arch, Bn, K, T, P = cfg["target"], cfg["batch"], cfg["K"], cfg["temperature"], cfg["prompt"]
    seeds = cfg["seeds"]
    t_dev = random_weights_on_device(arch, seeds["w"], torch, **late_scaling(cfg))
    target = B.Model(arch, t_dev)
    if isinstance(cfg["draft"], str):
        draft = target.share_prefix(int(cfg["draft"].split(":")[1]))
        d_dev = None
    else:
        d_dev = random_weights_on_device(cfg["draft"], seeds["wd"], torch)
        draft = B.Model(cfg["draft"], d_dev)
    steps, warm = args.steps, max(args.warmup, 3)
    prof_steps = min(steps, 16)
    n_it = steps + warm + prof_steps + 8          # iterations an engine may run (timed region + per-launch timing)
    max_len = P + n_it * (K + 1) + 16
    if arch.pos == 0:
        max_len = min(max_len, arch.max_pos)
    out_cap = n_it * (K + 1)
    prompts = torch.from_numpy(synth.gen_prompt(seeds["prompt"], Bn, P, arch.vocab)).cuda()

    def uniforms(n_iters, width):
        return np.stack([np.stack([synth.gen_uniforms(seeds["u"] + rank, s, it, width) for s in range(Bn)])
                         for it in range(n_iters)])  # [iters, B, width]

    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---------------- speculative: device-resident inputs ----------------
    eng = engine.Engine(target, draft, Bn, max_len, K, T, out_cap)
    eng.prefill(prompts)
    u_all = uniforms(warm + steps, 2 * K + 1)
    ud = torch.from_numpy(u_all[:, :, :K].copy()).cuda()
    uv = torch.from_numpy(u_all[:, :, K:].copy()).cuda()
    for it in range(warm):
        eng.spec_iteration(ud[it], uv[it])
        eng.advance()
    eng.refresh_bounds()
    barrier()
    count0 = eng.out_count.clone()
    launches0 = B.launch_count()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.profiler.start()   # lets a profiler run with --profile-from-start off see just this region
    e0.record()
    for it in range(warm, warm + steps):
        eng.spec_iteration(ud[it], uv[it])
        eng.advance()
    e1.record()
    barrier()
    torch.cuda.profiler.stop()
    spec_ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    launches = B.launch_count() - launches0
    spec_tokens = int((eng.out_count - count0).sum().item())
    accepted_mean = spec_tokens / (steps * Bn) - 1.0
    # per-token acceptance rate: accepted drafts / drafts that were tested (those up to and including the
    # first rejection of an iteration)
    acc_log = eng.n_acc_log[warm:warm + steps].cpu().numpy().ravel()
    hist = np.bincount(acc_log, minlength=K + 1).astype(np.int64)      # [K+1]: iterations with a accepted
    n_acc_tot = int((hist * np.arange(K + 1)).sum())
    n_tested = int((hist[:K] * (np.arange(K) + 1)).sum() + hist[K] * K)
    alpha = n_acc_tot / n_tested if n_tested else 0.0
    ctx_lens = eng.tkv.lengths()
    status = eng.tkv.status() or eng.dkv.status()

    # ---------------- dominant kernel (the forward kernel: draft forwards and verify passes)
    #                  timed with CUDA events around every launch over a repeat of the timed region ----
    B.gemm_profile(True)
    for it in range(warm, warm + prof_steps):    # (further iterations on the same engine: the caches have room)
        eng.spec_iteration(ud[it], uv[it])
        eng.advance()
    n_fwd, fwd_ms = B.gemm_profile_read()
    B.gemm_profile(False)
    d_arch = draft.arch
    p_lens = eng.tkv.lengths()
    # algorithmic bytes of those launches: K draft steps (draft matrices + draft KV) + one verify pass
    draft_step_bytes = verify_step_bytes(d_arch, Bn, 0, p_lens) - Bn * 4
    fwd_bytes = prof_steps * (verify_step_bytes(arch, Bn, K, p_lens) + K * draft_step_bytes)
    fwd_gbs = fwd_bytes / (fwd_ms * 1e-3) / 1e9 if fwd_ms > 0 else 0.0

    # ---------------- the draft loop alone: one draft_step call per token, and all K steps in one launch ----------------
    def time_draft(fused, reps):
        d_eng = engine.Engine(target, draft, Bn, max_len, K, T, 8)
        d_eng.copy_cache_from(eng)
        d_eng.dkv.buf.copy_(eng.dkv.buf)
        d_eng.draft_in.copy_(eng.draft_in)
        d_eng.draft_n_in.fill_(1)
        len0 = torch.from_numpy(d_eng.dkv.lengths()).cuda()
        d_eng.fused_draft = fused
        us = ud[0].stride(0)

        def loop():
            if fused:
                B.draft_steps(draft, d_eng.dkv, K, d_eng.draft_in, 2, 2, d_eng.draft_n_in, T, ud[0], us,
                              d_eng.rows[:, 1:], K + 1, d_eng.q, K * arch.vocab, d_eng.ws_d)
            else:
                for i in range(K):
                    if i == 0:
                        B.draft_step(draft, d_eng.dkv, d_eng.draft_in, 2, 2, d_eng.draft_n_in, T, ud[0], us,
                                     d_eng.rows[:, 1:], K + 1, d_eng.q[:, 0], K * arch.vocab, d_eng.ws_d)
                    else:
                        B.draft_step(draft, d_eng.dkv, d_eng.rows[:, i:], K + 1, 1, None, T, ud[0][:, i:], us,
                                     d_eng.rows[:, i + 1:], K + 1, d_eng.q[:, i], K * arch.vocab, d_eng.ws_d)
            B.kv_rollback(d_eng.dkv, len0)     # the same context every time
        for _ in range(2):
            loop()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            loop()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps / K

    draft_ms = {"per_token_calls_ms_per_step": time_draft(False, 5), "one_launch_ms_per_step": time_draft(True, 5),
                "algorithmic_bytes_per_step": verify_step_bytes(draft.arch, Bn, 0, eng.dkv.lengths()) - Bn * 4}

    # ---------------- verification pass alone, and one-row decode, on the same cache ----------------
    def time_verify(k, reps, e):
        q = eng.q[:, :max(k, 1)].contiguous() if k else None
        u = uv[0][:, :k + 1].contiguous()
        rows = eng.rows[:, :k + 1].contiguous()
        ws = e.ws_t
        for _ in range(3):
            B.target_verify(target, e.tkv, rows, k, q, u, T, eng.n_acc, eng.next_tok, 1, None, ws)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            B.target_verify(target, e.tkv, rows, k, q, u, T, eng.n_acc, eng.next_tok, 1, None, ws)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps, e.tkv.lengths()

    reps = max(5, min(steps, 20))
    verify_ms, v_lens = time_verify(K, reps, eng)
    # the verify launches of the forward kernel alone, CUDA events around each launch
    B.gemm_profile(True)
    time_verify(K, reps, eng)
    n_vf, vf_ms = B.gemm_profile_read()
    B.gemm_profile(False)
    v_bytes = verify_step_bytes(arch, Bn, K, v_lens)
    # the same cache, one row per sequence
    dec = engine.Engine(target, None, Bn, max_len, 0, T, out_cap)
    dec.copy_cache_from(eng)
    decode_ms, d_lens = time_verify(0, reps, dec)
    d_bytes = verify_step_bytes(arch, Bn, 0, d_lens)
    del eng, dec
    torch.cuda.empty_cache()

    # ---------------- autoregressive generation ----------------
    ar = engine.Engine(target, None, Bn, max_len, 0, T, out_cap)
    ar.prefill(prompts)
    u1 = torch.from_numpy(uniforms(warm + steps, 1)).cuda()
    for it in range(warm):
        ar.ar_step(u1[it])
    ar.refresh_bounds()
    barrier()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for it in range(warm, warm + steps):
        ar.ar_step(u1[it])
    a1.record()
    barrier()
    ar_ms = a0.elapsed_time(a1)
    ar_tps = steps * Bn / (ar_ms * 1e-3)
    del ar
    torch.cuda.empty_cache()

    # ---------------- end to end: host buffers, copies inside the timed region ----------------
    eng2 = engine.Engine(target, draft, Bn, max_len, K, T, out_cap)
    eng2.prefill(prompts)
    pin_ud = torch.from_numpy(np.ascontiguousarray(u_all[:, :, :K])).pin_memory()
    pin_uv = torch.from_numpy(np.ascontiguousarray(u_all[:, :, K:])).pin_memory()
    host_acc = torch.zeros(Bn, dtype=torch.int32).pin_memory()
    host_rows = torch.zeros(Bn, K + 1, dtype=torch.int32).pin_memory()
    host_next = torch.zeros(Bn, dtype=torch.int32).pin_memory()
    dev_ud = torch.zeros(Bn, K, device="cuda")
    dev_uv = torch.zeros(Bn, K + 1, device="cuda")
    for it in range(warm):
        eng2.spec_iteration(ud[it], uv[it])
        eng2.advance()
    eng2.refresh_bounds()
    barrier()
    c0 = eng2.out_count.clone()
    t0 = time.perf_counter()
    for it in range(warm, warm + steps):
        dev_ud.copy_(pin_ud[it], non_blocking=True)                     # H2D: this step's uniforms
        dev_uv.copy_(pin_uv[it], non_blocking=True)
        eng2.spec_iteration(dev_ud, dev_uv)
        host_acc.copy_(eng2.n_acc, non_blocking=True)                   # D2H: accepted count, draft tokens,
        host_rows.copy_(eng2.rows, non_blocking=True)                   #      the token drawn by the target
        host_next.copy_(eng2.next_tok, non_blocking=True)
        eng2.advance()
        torch.cuda.synchronize()
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_tokens = int((eng2.out_count - c0).sum().item())
    h2d = Bn * (2 * K + 1) * 4
    d2h = Bn * (K + 3) * 4
    del eng2
    torch.cuda.empty_cache()

    # ---------------- the verification pass at batch 1, context 2048 (7B shape only) ----------------
    vb1 = verify_batch1(target, arch, torch, B, synth, reps) if args.workload.startswith("llama-7b-b") else None

    # ---------------- the prompt pass (fills the cache before sampling starts) ----------------
    pp = prompt_pass(target, arch, torch, B, synth, Bn, min(P - 1, 1024), seeds["prompt"]) if arch.dtype and rank == 0 else None

    # ---------------- whole generations of 40 and 100 new tokens, as a caller times them ----------------
    wc = whole_call(engine, target, draft, Bn, K, T, prompts.cpu().numpy(), synth, seeds["u"] + 7, torch) if rank == 0 else None

    # ---------------- aggregate over ranks ----------------
    tot_tokens, tot_e2e_tokens, max_ms, max_e2e = aggregate_replicas(
        dist, [spec_tokens, e2e_tokens], [spec_ms, e2e_s], "cuda")

    peak, which = measured_hbm_peak()
    vf_gbs = v_bytes * n_vf / (vf_ms * 1e-3) / 1e9 if vf_ms > 0 else 0.0
    line = {
        "metric": METRIC, "value": tot_tokens / (max_ms * 1e-3), "unit": "tok/s", "n_gpus": world,
        "steps": steps, "warmup": warm, "ms_per_step": max_ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if arch.dtype else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "batch": Bn, "prompt": P, "K": K, "temperature": T,
                   "target": f"{arch.n_layers}L d{arch.d_model} V{arch.vocab}",
                   "draft": cfg["draft"] if isinstance(cfg["draft"], str) else
                   f"{cfg['draft'].n_layers}L d{cfg['draft'].d_model}",
                   "l2": "inputs larger than L2 (weights streamed each pass exceed 126 MB)",
                   "multi_gpu": "replicas only (independent sequences, no collective)"},
        "clocks": clocks,
        "e2e": {"value": tot_e2e_tokens / max_e2e, "unit": "tok/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        # the dominant kernel is forward_kernel (one launch per verify pass; the draft steps of an iteration
        # are launches of the same kernel); the figure is for its verify launches, the pass the method is
        # about; all launches of the timed region are given beside it
        "roofline": {"bound": "hbm", "achieved": vf_gbs, "peak": peak, "unit": "GB/s",
                     "frac": vf_gbs / peak, "traffic": scaled_traffic(args.workload, arch, Bn * (K + 1)),
                     "peak_source": which, "kernel": "forward_kernel (verify launches)", "launches": n_vf,
                     "avg_launch_us": 1e3 * vf_ms / max(n_vf, 1), "bytes_per_launch": v_bytes,
                     "frac_of_8tbs": vf_gbs / NOMINAL_HBM_GBS,
                     "all_launches": {"achieved": fwd_gbs, "frac": fwd_gbs / peak, "launches": n_fwd,
                                      "avg_launch_us": 1e3 * fwd_ms / max(n_fwd, 1),
                                      "bytes_per_launch_avg": fwd_bytes / max(n_fwd, 1)}},
        "speculative": {"tok_s": spec_tokens / (spec_ms * 1e-3), "accepted_per_iter": accepted_mean,
                        "tokens_per_iter": spec_tokens / (steps * Bn), "alpha": alpha,
                        "tokens_per_iter_closed_form": expected_tokens_per_iteration(alpha, K)},
        "autoregressive": {"tok_s": ar_tps, "ms_per_token": ar_ms / steps},
        "draft_loop": draft_ms,
        "verify": {"ms": verify_ms, "rows": Bn * (K + 1), "bytes": v_bytes, "gbs": v_bytes / verify_ms / 1e6,
                   "frac_of_peak": v_bytes / verify_ms / 1e6 / peak,
                   "frac_of_8tbs": v_bytes / verify_ms / 1e6 / NOMINAL_HBM_GBS,
                   "decode_ms": decode_ms, "decode_gbs": d_bytes / decode_ms / 1e6,
                   "verify_over_decode": verify_ms / decode_ms, "ctx": [int(x) for x in v_lens]},
        "device_status": int(status),
    }
    if vb1 is not None:
        line["verify_b1"] = vb1
    if pp is not None:
        line["prompt_pass"] = pp
    if wc is not None:
        line["whole_call"] = wc
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        host_w = (weights_to_host(t_dev, torch), None if d_dev is None else weights_to_host(d_dev, torch))
        del t_dev, d_dev, target, draft
        torch.cuda.empty_cache()
        line["cpu_baseline"] = cpu_baseline(args.workload, steps=None, budget_s=20.0, weights=host_w,
                                            single_thread=True)
    if dist is not None:
        dist.destroy_process_group()
    return line


def measured_bf16_peak():
    try:
        return float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"]), "measured"
    except Exception:
        return FALLBACK_BF16_TFLOPS, "fallback"


def prompt_pass(target, arch, torch, B, synth, Bn, P, seed):
    """The prompt pass that fills the cache (no logits): `Bn` sequences x `P` tokens through kv_prefill in its
    many-row form (tiled tcgen05 GEMMs; compute-bound, so the yardstick is the measured bf16 GEMM rate: the
    projections run every activation as bf16 hi + lo, twice the useful products) and in its few-row form
    (passes of the verification kernel, 64 rows each)."""
    S = P + 64
    prompts = torch.from_numpy(synth.gen_prompt(seed, Bn, P, arch.vocab)).cuda()
    lens = torch.full((Bn,), P, dtype=torch.int32, device="cuda")
    zero = torch.zeros(Bn, dtype=torch.int32, device="cuda")
    kv = B.KV(target, Bn, S)
    rows = min(P, 8192 // Bn)
    C = min(B.MAX_ROWS_PER_SEQ, B.MAX_ROWS // Bn)
    ms = {}
    for mode, reps in ((0, 3), (1, 2)):
        nbytes = max(target.prefill_workspace_bytes(Bn, rows) if mode == 0 else 0, target.workspace_bytes(Bn, C, S))
        ws = B.device_buffer(nbytes)
        B.set_prefill_mode(mode)
        try:
            ts = []
            for _ in range(reps):
                B.kv_rollback(kv, zero)
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                B.kv_prefill(target, kv, prompts, lens, ws)
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
        finally:
            B.set_prefill_mode(0)
        ms[mode] = (min(ts[1:]), nbytes)      # (the first repetition warms up)
        del ws
        torch.cuda.empty_cache()
    status = kv.status()
    d, F = arch.d_model, arch.d_ff
    useful = 2.0 * Bn * P * arch.n_layers * (3 * d * d + d * d + arch.d_in * d + d * F)
    peak, which = measured_bf16_peak()
    t = ms[0][0] * 1e-3
    return {"batch": Bn, "tokens_per_seq": P, "ms": ms[0][0], "tok_s": Bn * P / t, "workspace_bytes": ms[0][1],
            "rows_per_pass": Bn * rows, "few_row_form_ms": ms[1][0], "speedup_over_few_row_form": ms[1][0] / ms[0][0],
            "projection_tflops_useful": useful / t / 1e12, "projection_tflops_tensor": 2 * useful / t / 1e12,
            "bf16_peak_tflops": peak, "peak_source": which + " (sustained cuBLAS bf16)",
            "frac_of_bf16_peak": 2 * useful / t / 1e12 / peak, "device_status": int(status)}


def whole_call(engine, target, draft, Bn, K, T, prompts_np, synth, seed, torch, n_list=(40, 100)):
    """Wall-clock time of whole generations as a caller sees them - prompt pass, iterations until every sequence
    has N new tokens, host polling of the counters included - for N = 40 and 100 new tokens, speculative and
    autoregressive (the quantity the paper's Table of timings reports per prompt)."""
    P = prompts_np.shape[1]
    out = {"prompt_tokens": P, "n_new": list(n_list), "speculative_s": [], "autoregressive_s": [], "iterations": []}
    for N in n_list:
        for k, dm, key in ((K, draft, "speculative_s"), (0, None, "autoregressive_s")):
            max_len = P + (N + 8) * (k + 1) + 16
            if target.arch.pos == 0:
                max_len = min(max_len, target.arch.max_pos)
            eng = engine.Engine(target, dm, Bn, max_len, k, T, (N + 8) * (k + 1))
            width = 2 * k + 1
            u = lambda s_, it: synth.gen_uniforms(seed, s_, it, width)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            res = eng.generate(prompts_np, N, u)
            torch.cuda.synchronize()
            out[key].append(time.perf_counter() - t0)
            if k:
                out["iterations"].append(int(res["iterations"]))
            del eng
            torch.cuda.empty_cache()
    out["speedup"] = [a / s for a, s in zip(out["autoregressive_s"], out["speculative_s"])]
    return out


def run_prompt_pass(args):
    """The prompt pass alone: the workload's target, its batch, --prompt-pass tokens per sequence."""
    import torch
    from paper_2311_04951_b200 import binding as B, synth
    torch.cuda.set_device(0)
    cfg = resolve(args.workload)
    arch = cfg["target"]
    target = B.Model(arch, random_weights_on_device(arch, cfg["seeds"]["w"], torch, **late_scaling(cfg)))
    out = prompt_pass(target, arch, torch, B, synth, cfg["batch"], args.prompt_pass, cfg["seeds"]["prompt"])
    out["workload"] = args.workload
    return out


def verify_batch1(target, arch, torch, B, synth, reps, ctx=2048, rows_list=(1, 4, 5)):
    """One sequence, `ctx` cached positions (seeded N(0,1) fill), verification passes over 1, 4 and 5 rows:
    latency, algorithmic GB/s, fraction of the HBM peak, and the ratio to the one-row pass."""
    peak, _ = measured_hbm_peak()
    S = ctx + 64
    kv = B.KV(target, 1, S)
    g = torch.Generator(device="cuda")
    g.manual_seed(41 + ctx)
    kv.cache_view().copy_(torch.randn(kv.cache_view().shape, generator=g, device="cuda", dtype=torch.float32))
    B.kv_commit(kv, torch.tensor([ctx], dtype=torch.int32, device="cuda"))
    kv.lengths()
    V = arch.vocab
    out = {"ctx": ctx, "points": []}
    for M in rows_list:
        K = M - 1
        ws = target.new_workspace(1, M, S)
        rows = torch.from_numpy(synth.gen_prompt(42, 1, M, V)).cuda()
        q = torch.from_numpy(synth.gen_dirichlet_rows(43, max(K, 1), V)).cuda().reshape(1, max(K, 1), V)
        u = torch.from_numpy(synth.gen_uniforms(44, 0, 0, M)).cuda().reshape(1, M)
        na = torch.zeros(1, dtype=torch.int32, device="cuda")
        nx = torch.zeros(1, dtype=torch.int32, device="cuda")
        call = lambda: B.target_verify(target, kv, rows, K, q if K else None, u, 1.0, na, nx, 1, None, ws)
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        ts = []
        for _ in range(max(reps, 10)):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            call()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ms = float(np.median(ts))
        nbytes = verify_step_bytes(arch, 1, K, [ctx])
        out["points"].append({"rows": M, "ms": ms, "bytes": nbytes, "gbs": nbytes / ms / 1e6,
                              "frac_of_peak": nbytes / ms / 1e6 / peak,
                              "frac_of_8tbs": nbytes / ms / 1e6 / NOMINAL_HBM_GBS})
    base = out["points"][0]["ms"]
    for pt in out["points"]:
        pt["verify_over_decode"] = pt["ms"] / base
    return out


def aggregate_replicas(dist, sums, maxima, device):
    """Replicas only: every rank generates for its own sequences, no data-path collective.  The job's
    tokens are the SUM over ranks, its time is the MAX over ranks.  `dist` is torch.distributed (an
    initialised process group) or None for a single process."""
    if dist is None:
        return [*sums, *maxima]
    import torch
    t = torch.tensor([float(x) for x in sums], dtype=torch.float64, device=device)
    m = torch.tensor([float(x) for x in maxima], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return [*(int(round(x)) for x in t.tolist()), *m.tolist()]


# ------------------------------------------------------------------ isolated verify sweep
def run_sweep(args):
    """Isolated verification-pass sweep at the 7B Llama shape: rows in {1,2,3,4,5,8,9,16,17} x cache
    context in {512, 2048, 8192, 16384}, batch 1; cache filled with seeded N(0,1) values, draft rows
    Dirichlet(0.1).  Prints one JSON object with latency, GB/s and fraction of the HBM peak per point."""
    import torch
    from paper_2311_04951_b200 import binding as B, synth
    torch.cuda.set_device(0)
    arch = synth.PRESETS["llama-7b"]["target"]
    target = B.Model(arch, random_weights_on_device(arch, 31, torch))
    peak, which = measured_hbm_peak()
    points = []
    for ctx in (512, 2048, 8192, 16384):
        r = verify_batch1(target, arch, torch, B, synth, max(args.steps, 10), ctx=ctx,
                          rows_list=(1, 2, 3, 4, 5, 8, 9, 16, 17))
        for pt in r["points"]:
            pt["ctx"] = ctx
            pt["over_one_row"] = pt.pop("verify_over_decode")
            points.append(pt)
    return {"sweep": "verify pass, llama-7b shape, batch 1", "peak_gbs": peak, "peak_source": which, "points": points}


# ------------------------------------------------------------------ CPU oracle timing
def oracle_weights(cfg):
    """Host arrays for the oracle's target and draft.  The large shapes are drawn on the GPU when there is
    one (seconds instead of minutes for 7 x 10^9 normal deviates) and copied back as data."""
    from paper_2311_04951_b200 import synth
    arch = cfg["target"]
    big = arch.n_layers * arch.d_model * arch.d_model > (1 << 28)
    try:
        import torch
        on_gpu = big and torch.cuda.is_available()
    except Exception:
        on_gpu = False
    if on_gpu:
        torch.cuda.set_device(0)
        tw = weights_to_host(random_weights_on_device(arch, cfg["seeds"]["w"], torch, **late_scaling(cfg)), torch)
        dw = None
        if not isinstance(cfg["draft"], str):
            dw = weights_to_host(random_weights_on_device(cfg["draft"], cfg["seeds"]["wd"], torch), torch)
        torch.cuda.empty_cache()
        return tw, dw
    tw = synth.gen_weights(arch, cfg["seeds"]["w"], **late_scaling(cfg))
    dw = None if isinstance(cfg["draft"], str) else synth.gen_weights(cfg["draft"], cfg["seeds"]["wd"])
    return tw, dw


def cpu_baseline(workload, steps, budget_s, warmup=0, weights=None, single_thread=False):
    """The oracle as it stands, on the host cores: speculative iterations of the same models (same
    shapes and init), ONE sequence from a SHORT prompt (16 tokens), timed whole.  With single_thread,
    one verification pass of the target (K+1 rows) is also timed on one core."""
    from oracle import decoder as od, sampling as osamp
    from paper_2311_04951_b200 import synth
    cfg = resolve(workload)
    arch, K, T = cfg["target"], cfg["K"], cfg["temperature"]
    cores = os.cpu_count() or 1
    od.set_threads(cores)
    tw, dw = weights if weights is not None else oracle_weights(cfg)
    tgt = od.Model(arch, tw)
    if isinstance(cfg["draft"], str):
        d_arch, d_ws = synth.prefix_draft(arch, tw, int(cfg["draft"].split(":")[1]))
    else:
        d_arch, d_ws = cfg["draft"], dw
    drf = od.Model(d_arch, d_ws)
    P = 16
    prompt = synth.gen_prompt(cfg["seeds"]["prompt"], 1, P, arch.vocab)[0]
    s_max = P + 64 * (K + 1)
    if arch.pos == 0:
        s_max = min(s_max, arch.max_pos)
    tc, dc = tgt.new_cache(s_max), drf.new_cache(s_max)
    tc.feed(prompt[:-1], want_logits=False)
    dc.feed(prompt[:-1], want_logits=False)
    x = [int(t) for t in prompt]
    tokens, iters, t0 = 0, -int(warmup), time.perf_counter()
    t_start = t0
    while True:
        u = synth.gen_uniforms(cfg["seeds"]["u"], 0, iters + int(warmup), 2 * K + 1)
        n = len(x)
        feed, qs, drafts = x[dc.len:n], [], []
        for i in range(K):
            q = osamp.softmax_t(dc.feed(feed)[-1], T)
            t = osamp.inv_cdf(q, u[i])
            qs.append(q)
            drafts.append(t)
            feed = [t]
        lg = tc.feed([x[n - 1]] + drafts, advance=False)
        ps = [osamp.softmax_t(lg[i], T) for i in range(K + 1)]
        a, y = osamp.accept_resample(ps, qs, drafts, u[K:2 * K], u[2 * K])
        x.extend(drafts[:a] + [y])
        tc.len += a + 1
        dc.rollback(min(n + a, n + K - 1))
        iters += 1
        if iters <= 0:  # an untimed warm-up iteration: the clock and the token count start behind it
            if iters == 0:
                t0 = time.perf_counter()
            continue
        tokens += a + 1
        el = time.perf_counter() - t0
        if (steps is not None and iters >= steps) or time.perf_counter() - t_start > budget_s or \
                (steps is None and iters >= 32) or tc.len + 2 * (K + 1) > s_max:
            break
    out = {"value": tokens / el, "unit": "tok/s", "cores": od.get_threads(), "kind": "oracle",
           "sample": f"{iters} speculative iteration(s) of the {workload} models, ONE sequence (batch 1), prompt {P}, "
                     f"K={K}, {tokens} tokens in {el:.1f} s",
           "ms_per_step": 1e3 * el / iters, "iters": iters}
    if single_thread:
        od.set_threads(1)
        t1 = time.perf_counter()
        tc.feed([x[-1]] * (K + 1), advance=False)
        dt = time.perf_counter() - t1
        od.set_threads(cores)
        out["single_thread"] = {"verify_pass_s": dt, "rows": K + 1, "cores": 1,
                                "sample": f"one verification pass of the target, {K + 1} rows, context {tc.len}"}
    return out


def run_reference(args, rank, world):
    """Reference arm = the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return None
    cb = cpu_baseline(args.workload, steps=args.steps, budget_s=150.0, warmup=min(max(args.warmup, 0), 1))
    cfg = resolve(args.workload)
    arch = cfg["target"]
    return {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": "tok/s", "n_gpus": world,
            "steps": cb["iters"], "warmup": min(max(args.warmup, 0), 1), "ms_per_step": cb["ms_per_step"],
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 storage, f64 accumulate", "data": "synthetic",
            "config": {"workload": args.workload, "batch": 1, "prompt": 16, "K": cfg["K"],
                       "temperature": cfg["temperature"], "target": f"{arch.n_layers}L d{arch.d_model} V{arch.vocab}"},
            "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
            "e2e": {"value": cb["value"], "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


# ------------------------------------------------------------------ launcher
def replica_command(args, argv, port):
    """The command that runs this script as `args.gpus` replica processes on one node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_replicas(args, argv):
    """--gpus N > 1 without a launcher around us: start N ranks of this script and pass their output on."""
    if args.impl == "ours":
        import torch
        n = torch.cuda.device_count()
        if n < args.gpus:
            raise SystemExit(f"bench.py --gpus {args.gpus}: only {n} GPU(s) visible")
    return subprocess.call(replica_command(args, argv, free_port()))


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="isolated verify-pass sweep at the 7B shape (one GPU)")
    ap.add_argument("--prompt-pass", type=int, default=0, metavar="TOKENS",
                    help="only the prompt pass of the workload's target: batch x TOKENS tokens (one GPU)")
    args = ap.parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.sweep and not args.prompt_pass:
        return launch_replicas(args, argv)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.sweep:
        line = run_sweep(args) if rank == 0 else None
    elif args.prompt_pass:
        line = run_prompt_pass(args) if rank == 0 else None
    elif args.impl == "reference":
        line = run_reference(args, rank, world)
    else:
        line = run_ours(args, rank, world)
    if rank == 0 and line is not None:
        print(json.dumps(line), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
