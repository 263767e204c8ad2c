#!/usr/bin/env python
"""Benchmark of the Spec-VLA tree-verification path on B200.

One step = one action chunk of the C1 workload (OpenVLA-7B-shaped decoder, batch 1,
290-position prefix, 26-node draft tree from the one-layer draft model, 7 action tokens,
strict acceptance r = 0) through specvla_generate_action: prefill, then draft -> verify ->
accept -> compact until 7 tokens. Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 runs N independent replicas (one process per GPU under torchrun); there is no
data-path collective because episodes are independent.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "action chunks/sec at bs1 (7B)"
UNIT = "chunks/s"
WEIGHT_BYTES_PER_VERIFY = 13_214_679_040      # 32 layers + LM head, bf16, read once


# DRAM traffic of one gate/up launch at T = 27 from the ncu capture under profiles/ (bytes); to be
# re-taken (or set to None) whenever gemm_ck.cuh changes.
GATE_UP_DRAM_BYTES = 203_328_256 + 5_499_136


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained"), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    samples=len(sm), reasons=sorted(reasons))


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_sample(device, iters_per_chunk: int, depth: int, pieces=None):
    """Times the oracle, as it stands, on a bounded slice of the C1 chunk and extrapolates.

    Slice: one target decoder layer over the 290 prefix rows, one over the 27 tree rows, the LM
    head over 27 rows and one draft-model level (fc + layer + LM head + log-softmax) over 4
    rows, all at the 7B shapes. chunk_est = 33 t_layer(290) + iters * (32 t_layer(27) +
    t_lm(27) + depth * t_draft_level). Returns (chunks/s estimate, seconds used, pieces).
    `pieces` carries the terms measured by an earlier call that are not re-measured."""
    import torch
    from oracle import decoder as D
    from synth_inputs import configs as C, rng

    desc = C.OPENVLA_7B
    st = _oracle_state(device)
    w, T, P = st["w"], 27, 290
    t0 = time.perf_counter()
    out = dict(pieces or {})

    def timed(name, fn):
        if name in out and pieces is not None and name not in ("layer27", "lm27"):
            return
        a = time.perf_counter()
        fn()
        out[name] = time.perf_counter() - a

    def layer(rows, n_before):
        x = st["x"][:rows]
        cache = D.KVCache(1, n_before + rows, desc.n_heads, desc.head_dim)
        pos = torch.arange(n_before, n_before + rows)
        vis = torch.ones(rows, n_before + rows, dtype=torch.bool)
        D.decoder_layer(w, "layers.0.", desc, x, pos, pos, vis, cache, 0)

    def draft_level():
        cache = D.KVCache(1, P + 4, desc.n_heads, desc.head_dim)
        pos = torch.arange(P, P + 4)
        g = D.draft_forward(w, desc, st["x"][:4], st["x"][4:8], pos, pos,
                            torch.ones(4, P + 4, dtype=torch.bool), cache)
        torch.log_softmax(D.lm_head(w, g)[:, desc.action_base:desc.action_base + desc.n_bins], dim=1)

    timed("layer290", lambda: layer(P, 0))
    timed("layer27", lambda: layer(T, P))
    timed("lm27", lambda: D.lm_head(w, st["x"][:T]))
    timed("draft_level", draft_level)
    chunk = 33 * out["layer290"] + iters_per_chunk * (32 * out["layer27"] + out["lm27"] +
                                                     depth * out["draft_level"])
    return 1.0 / chunk, time.perf_counter() - t0, out


_ORACLE_STATE = {}


def _oracle_state(device):
    if not _ORACLE_STATE:
        import torch
        from oracle import decoder as D
        from synth_inputs import configs as C, rng
        desc = C.OPENVLA_7B
        d, F, hd = desc.d_model, desc.d_ffn, desc.n_heads * desc.head_dim
        raw = {}

        def mat(stream, r, c):
            return rng.normal_bf16(1, stream, (r, c), 0.02, device).cpu()

        for prefix, base in (("layers.0.", C.STREAM_LAYER0), ("draft.layer.", C.STREAM_DRAFT_LAYER)):
            raw[prefix + "wqkv"] = torch.cat([mat(base + i, hd, d) for i in range(3)])
            raw[prefix + "wo"] = mat(base + 3, d, hd)
            raw[prefix + "wgu"] = torch.cat([mat(base + 4, F, d), mat(base + 5, F, d)])
            raw[prefix + "wd"] = mat(base + 6, d, F)
            raw[prefix + "norm1"] = torch.ones(d)
            raw[prefix + "norm2"] = torch.ones(d)
        raw["lm_head"] = mat(C.STREAM_LM_HEAD, desc.vocab, d)
        raw["draft.fc"] = mat(C.STREAM_DRAFT_FC, d, 2 * d)
        _ORACLE_STATE["w"] = D.DecoderWeights(raw)
        _ORACLE_STATE["x"] = rng.normal(1, 999, (290, d), 1.0, "cpu")
    return _ORACLE_STATE


def run_reference(args, rank, world):
    """The reference arm: there is no reference implementation, so the CPU oracle is timed."""
    if rank != 0:
        return
    import torch
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    torch.set_grad_enabled(False)
    iters, depth = 6, 5
    pieces, times = None, []
    total = args.warmup + args.steps
    full_every_step = total * 10.0 <= 240.0
    for i in range(total):
        val, sec, pieces_new = oracle_sample(dev, iters, depth, None if (full_every_step or i == 0) else pieces)
        pieces = pieces_new
        if i >= args.warmup:
            times.append((val, sec))
    value = statistics.mean(v for v, _ in times)
    cores = torch.get_num_threads()
    sample = ("per step: oracle decoder layer over 290 and over 27 rows, LM head over 27 rows"
              + (", one draft level over 4 rows" if full_every_step else
                 " (290-row layer and draft level measured once in warm-up)")
              + "; chunk = 33*t_layer290 + 6*(32*t_layer27 + t_lm27 + 5*t_draft); 7B shapes, float64")
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1000.0 / value, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload="C1-openvla7b-bs1", prefix=290, tree_rows=27, n_tokens=7, r=0),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- replicas
def max_over_ranks(values, device, world):
    """Each value's maximum over the ranks of the job: N GPUs run N independent replicas, and a
    timed region lasts as long as its slowest replica. No other data crosses ranks."""
    if world == 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def replica_throughput(world, steps, ms):
    """Whole-job chunks/s: every rank finished `steps` chunks within `ms` (the slowest rank's time)."""
    return world * steps / (ms / 1000.0)


# --------------------------------------------------------------------------- CUDA arm
def run_ours(args, rank, local_rank, world):
    import torch
    import torch.distributed as dist
    from paper_2507_22424_b200.binding import SpecVLA, make_shape
    from synth_inputs import configs as C, data

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    wl, desc = C.C1, C.OPENVLA_7B
    weights = data.make_weights(desc, wl.seed, device="cuda")
    embeds, ids = data.make_prefix(wl, device="cuda")
    ids_host = ids.tolist()
    P = len(ids_host)
    gpu = SpecVLA(desc, weights, max_seq=512, max_episodes=1, max_rows=512, action_only=True)
    shape = make_shape(wl.tree.branch, wl.tree.expand)
    r, n_tok = 0, wl.n_tokens

    def chunk():
        return gpu.generate_action([0], embeds, ids_host, [P], shape, r, n_tok)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        toks, _, stats = chunk()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    # --- timed region 1: inputs resident in HBM -----------------------------------------
    barrier()
    l0 = gpu.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ms_verify = ms_draft = ms_prefill = 0.0
    iters = accept = 0
    for _ in range(args.steps):
        toks, _, stats = chunk()
        ms_verify += stats.ms_verify
        ms_draft += stats.ms_draft
        ms_prefill += stats.ms_prefill
        iters += stats.iterations
        accept += sum(stats.accept_len[i] for i in range(min(16, stats.iterations)))
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = gpu.kernel_launches() - l0
    clocks = sampler.stop() if rank == 0 else None
    # --- timed region 2: end to end from host buffers ----------------------------------
    embeds_host = embeds.cpu().pin_memory()
    stage = torch.empty_like(embeds)
    barrier()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for _ in range(args.steps):
        stage.copy_(embeds_host, non_blocking=True)
        toks_e2e, acts, _ = gpu.generate_action([0], stage, ids_host, [P], shape, r, n_tok)
    e3.record()
    barrier()
    ms_e2e = e2.elapsed_time(e3)
    # --- AR baseline from the same kernels (depth-0 tree) --------------------------------
    ar_shape = make_shape((), ())
    gpu.generate_action([0], embeds, ids_host, [P], ar_shape, 0, n_tok)
    barrier()
    e4, e5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e4.record()
    ar_steps = max(3, args.steps // 2)
    ar_ms_verify = 0.0
    for _ in range(ar_steps):
        ar_toks, _, ar_stats = gpu.generate_action([0], embeds, ids_host, [P], ar_shape, 0, n_tok)
        ar_ms_verify += ar_stats.ms_verify
    e5.record()
    barrier()
    ms_ar = e4.elapsed_time(e5)
    # --- depth pruning: an iteration drafts no deeper than the tokens still missing ------------
    pr_shape = make_shape(wl.tree.branch, wl.tree.expand, prune=True)
    gpu.generate_action([0], embeds, ids_host, [P], pr_shape, r, n_tok)
    barrier()
    e6, e7 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e6.record()
    for _ in range(ar_steps):
        pr_toks, _, pr_stats = gpu.generate_action([0], embeds, ids_host, [P], pr_shape, r, n_tok)
    e7.record()
    barrier()
    ms_pr = e6.elapsed_time(e7)
    # --- the paper's dynamic tree: top-8, depth 5, best 50 of the 264 drafted nodes verified ----
    dy_shape = make_shape((8,) * 5, (1, 8, 8, 8, 8), keep=50)
    gpu.generate_action([0], embeds, ids_host, [P], dy_shape, r, n_tok)
    barrier()
    e8, e9 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e8.record()
    for _ in range(ar_steps):
        dy_toks, _, dy_stats = gpu.generate_action([0], embeds, ids_host, [P], dy_shape, r, n_tok)
    e9.record()
    barrier()
    ms_dy = e8.elapsed_time(e9)
    # --- perfect drafts: the same loop when the tree's first-child chain is the target's own greedy
    # continuation (known from the chunk just decoded), every other node a wrong token. The draft
    # model still runs and is paid for; its tree is replaced before verification. An upper bound of
    # what acceptance can buy on this workload (random draft weights accept nothing).
    t_par, t_dep = data.static_topology(wl.tree)
    chain = [0]
    for l in range(wl.tree.depth):
        chain.append(next(i for i in range(len(t_par)) if t_par[i] == chain[-1]))

    def perfect_chunk():
        first = gpu.prefill([0], embeds, ids_host, [P])
        out, its = [first[0]], 0
        while len(out) < n_tok:
            gpu.draft_tree([0], shape, want_trees=False)
            tok = [-1] + [desc.action_base + (17 * i) % desc.n_bins for i in range(1, len(t_par))]
            for j in range(1, len(chain)):
                want = toks[0][len(out) - 1 + j] if len(out) - 1 + j < n_tok else None
                for i in range(1, len(t_par)):            # no sibling may carry the right token
                    if t_dep[i] == j and tok[i] == want:
                        tok[i] = desc.action_base + (tok[i] - desc.action_base + 1) % desc.n_bins
                if want is not None:
                    tok[chain[j]] = want
            m, em = gpu.verify_tree([0], [dict(tokens=tok, parent=t_par, depth=t_dep)], r)
            out += em[0][:m[0] + 1]
            its += 1
        return out[:n_tok], its

    pf_toks, pf_its = perfect_chunk()
    barrier()
    e10, e11 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e10.record()
    for _ in range(ar_steps):
        pf_toks, pf_its = perfect_chunk()
    e11.record()
    barrier()
    ms_pf = e10.elapsed_time(e11)
    # --- per-GEMM device time of the verification phase (separate pass, same steps) -----
    gpu.profile(4)
    for _ in range(max(2, args.steps // 4)):
        chunk()
    prof = gpu.profile_read()
    gpu.profile(0)

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], "cuda", world)
    if rank != 0:
        gpu.close()
        dist.destroy_process_group()
        return
    peaks = load_peaks()
    value = replica_throughput(world, args.steps, ms)
    e2e_value = replica_throughput(world, args.steps, ms_e2e)
    T = 1 + wl.tree.n_nodes
    verify_ms = ms_verify / max(1, iters)
    kv_bytes = desc.n_layers * 2 * (P + 3 + T) * desc.d_model * 2 + T * desc.n_layers * 2 * desc.d_model * 2
    verify_gbs = (WEIGHT_BYTES_PER_VERIFY + kv_bytes) / (verify_ms * 1e-3) / 1e9
    dom = prof["gate_up"]
    N, K = 2 * desc.d_ffn, desc.d_model
    alg_bytes = N * K * 2 + T * K * 2 + T * N * 4
    dom_ms = dom["ms"] / max(1, dom["launches"])
    achieved = alg_bytes / (dom_ms * 1e-3) / 1e9 if dom["launches"] else None
    all_ms = sum(v["ms"] for v in prof.values())
    all_bytes = sum(v["bytes"] for v in prof.values())
    ipc = max(1, round(iters / args.steps))
    vals, cpu_sec, reps = [], 0.0, 0
    oracle_sample("cuda", ipc, wl.tree.depth)                      # untimed: page-in, thread pool
    while cpu_sec < 10.0 and reps < 64:
        v, sec, pieces = oracle_sample("cuda", ipc, wl.tree.depth)
        vals.append(v)
        cpu_sec += sec
        reps += 1
    cpu_val = statistics.mean(vals)
    line = dict(
        metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="bf16", data="synthetic",
        config=dict(workload=wl.name, prefix=P, tree_rows=T, tree="26 nodes depth 5 top-4/2/2/1/1",
                    n_tokens=n_tok, r=r, action_only=1, replicas=world,
                    l2="inputs larger than L2: every step streams 13.9 GB of weights"),
        e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=embeds.numel() * 2 + 4 * P,
                 d2h_bytes_per_step=4 * n_tok * 2 + 8 * max(1, round(iters / args.steps)) * 10),
        gpu_launches=launches,
        clocks=clocks,
        roofline=dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                      frac=(achieved / peaks["hbm_gbs"]) if achieved else None, traffic=GATE_UP_DRAM_BYTES,
                      traffic_source="ncu dram__bytes_read.sum + dram__bytes_write.sum of this launch "
                                     "(profiles/gemm_ck_verify_T27_ncu_full.md); the ~20 MB above the weights "
                                     "are the L2 prefetch of the next GEMM's weights",
                      kernel="weight-streaming GEMM, gate/up projection [22016 x 4096] at T=27 (verify)",
                      algorithmic_bytes_per_launch=alg_bytes, launches_timed=dom["launches"],
                      ms_per_launch=dom_ms, peak_source=peaks["source"] + " copy bandwidth",
                      all_verify_gemms_gbs=(all_bytes / (all_ms * 1e-3) / 1e9) if all_ms else None,
                      per_class={k: dict(ms_per_launch=v["ms"] / max(1, v["launches"]),
                                         gbs=(v["bytes"] / (v["ms"] * 1e-3) / 1e9) if v["ms"] else None)
                                 for k, v in prof.items()}),
        verify=dict(ms_per_step=verify_ms, hbm_gbs=verify_gbs, frac_of_measured_peak=verify_gbs / peaks["hbm_gbs"],
                    frac_of_8tbs=verify_gbs / 8000.0, bytes=WEIGHT_BYTES_PER_VERIFY + kv_bytes),
        phases_ms_per_chunk=dict(prefill=ms_prefill / args.steps, draft=ms_draft / args.steps,
                                 verify=ms_verify / args.steps),
        accept=dict(iterations_per_chunk=iters / args.steps, mean_m=accept / max(1, iters),
                    mean_tokens_per_forward=accept / max(1, iters) + 1.0),
        ar_baseline=dict(value=world * ar_steps / (ms_ar / 1000.0), unit=UNIT,
                         ms_per_decode_step=ar_ms_verify / (ar_steps * (n_tok - 1)),
                         same_tokens=bool(ar_toks == toks)),
        depth_pruned=dict(value=world * ar_steps / (ms_pr / 1000.0), unit=UNIT, same_tokens=bool(pr_toks == toks),
                          note="same call with tree_shape.prune = 1 (not Algorithm 1 as printed: iterations "
                               "draft min(depth, missing tokens - 1) levels); `value` above is unpruned"),
        perfect_drafts=dict(value=world * ar_steps / (ms_pf / 1000.0), unit=UNIT, iterations_per_chunk=pf_its,
                            same_tokens=bool(pf_toks == toks[0]),
                            note="the draft model runs, but the verified tree carries the target's own greedy "
                                 "continuation on its first-child chain: the ceiling acceptance could reach here"),
        dynamic_tree=dict(value=world * ar_steps / (ms_dy / 1000.0), unit=UNIT, same_tokens=bool(dy_toks == toks),
                          note="top-8, depth 5, best 50 of 264 drafted nodes verified (51 rows per step)"),
        cpu_baseline=dict(value=cpu_val, unit=UNIT, cores=torch.get_num_threads(), kind="oracle",
                          sample=("oracle (float64) decoder layer over 290 and 27 rows, LM head over 27 "
                                  "rows, one draft level over 4 rows at 7B shapes; chunk = 33*t_layer290 + "
                                  "iters*(32*t_layer27 + t_lm27 + 5*t_draft); mean of %d repetitions, %.1f s of CPU work"
                                  % (reps, cpu_sec)),
                          pieces_s=pieces),
        tokens=toks[0],
    )
    print(json.dumps(line), flush=True)
    gpu.close()
    if world > 1:
        dist.destroy_process_group()



# --------------------------------------------------------------------------- kernel micro-run
def run_micro(spec: str, steps: int, warmup: int):
    """`--micro gemm:T:N:K[:M]`: the stand-alone weight-streaming GEMM (specvla_gemm) over M
    distinct weight matrices in turn (default: enough to exceed the 126 MB L2 twice), timed
    with CUDA events per launch. One JSON line; the target of the ncu captures under profiles/."""
    import torch
    from paper_2507_22424_b200 import binding as B
    from synth_inputs import rng
    f = spec.split(":")
    if f[0] == "verify":
        return run_micro_verify(int(f[1]), int(f[2]) if len(f) > 2 else 27, steps, warmup,
                                persistent=(int(f[3]) if len(f) > 3 else 1))
    if f[0] == "batch":
        return run_micro_batch(int(f[1]) if len(f) > 1 else 16, steps, warmup)
    assert f[0] == "gemm" and len(f) in (4, 5), spec
    T, N, K = int(f[1]), int(f[2]), int(f[3])
    wbytes = N * K * 2
    M = int(f[4]) if len(f) == 5 else max(2, -(-2 * 126_000_000 // wbytes) + 1)
    torch.cuda.set_device(0)
    ws = [rng.normal_bf16(5, 10 + i, (N, K), 0.02, "cuda") for i in range(M)]
    x = rng.normal(5, 1, (T, K), 1.0, "cuda", dtype=torch.float32)
    g = B.GemmRunner(T, N, K)
    for i in range(warmup):
        g(x, ws[i % M])
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i, (a, b) in enumerate(ev):
        a.record()
        g(x, ws[(warmup + i) % M])
        b.record()
    torch.cuda.synchronize()
    ms = sorted(a.elapsed_time(b) for a, b in ev)
    med = ms[len(ms) // 2]
    peaks = load_peaks()
    alg = wbytes + T * K * 4 + T * N * 4
    print(json.dumps(dict(micro="gemm", T=T, N=N, K=K, matrices=M, steps=steps, ms_median=med, ms_min=ms[0],
                          note="whole specvla_gemm call: limb split + GEMM + plane sum",
                          algorithmic_bytes=alg, gbs_median=alg / med / 1e6, gbs_best=alg / ms[0] / 1e6,
                          frac_of_peak=alg / med / 1e6 / peaks["hbm_gbs"], peak=peaks["hbm_gbs"],
                          peak_source=peaks["source"])), flush=True)


def run_micro_verify(n_layers: int, rows: int, steps: int, warmup: int, persistent: int = 1):
    """`--micro verify:L[:T[:P]]` (P = 0: one launch per GEMM instead of the persistent forward kernel): verification steps of a 7B-SHAPED decoder cut down to L layers (a few
    GB on the device instead of 28), random T-row trees, strict acceptance. The small case of the
    real kernels (repacked weights, fused epilogues, PDL) for ncu --set full captures; also prints
    the per-GEMM device times of the verification phase."""
    import dataclasses
    import torch
    from paper_2507_22424_b200.binding import SpecVLA
    from synth_inputs import configs as C, data
    torch.cuda.set_device(0)
    desc = dataclasses.replace(C.OPENVLA_7B, n_layers=n_layers)
    wl = dataclasses.replace(C.C1, model=desc)
    weights = data.make_weights(desc, wl.seed, device="cuda", with_draft=False)
    embeds, ids = data.make_prefix(wl, device="cuda")
    ids_host, P = ids.tolist(), len(ids)
    gpu = SpecVLA(desc, weights, max_seq=1024, max_episodes=1, max_rows=512, action_only=True)
    from paper_2507_22424_b200.binding import OPT_PERSISTENT_FORWARD
    gpu.set_option(OPT_PERSISTENT_FORWARD, persistent)
    first = gpu.prefill([0], embeds, ids_host, [P])
    trees = []
    for i in range(warmup + steps):
        tok, par, dep = data.random_tree(rows, desc, seed=2, max_depth=8, stream_offset=10 * i)
        trees.append(dict(tokens=[-1] + tok[1:], parent=par, depth=dep))
    for i in range(warmup):
        gpu.verify_tree([0], [trees[i]], 0)
    gpu.profile(4)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(steps):
        gpu.verify_tree([0], [trees[warmup + i]], 0)
    b.record()
    torch.cuda.synchronize()
    prof = gpu.profile_read()
    ms = a.elapsed_time(b) / steps
    wbytes = n_layers * 404_750_336 + 262_668_288
    print(json.dumps(dict(micro="verify", layers=n_layers, rows=rows, steps=steps, persistent=persistent, ms_per_step=ms,
                          weight_bytes=wbytes, gbs=wbytes / ms / 1e6,
                          note="ms_per_step includes the per-GEMM timing events and the host read-back",
                          per_class={k: dict(us_per_launch=1e3 * v["ms"] / max(1, v["launches"]),
                                             gbs=(v["bytes"] / (v["ms"] * 1e-3) / 1e9) if v["ms"] else None)
                                     for k, v in prof.items()})), flush=True)
    gpu.close()


def run_micro_batch(n_ep: int, steps: int, warmup: int):
    """`--micro batch[:E]`: the batched workload (C4: E ragged episodes of 276-316 prefix rows, 27-row
    random trees, r = 4) on the full 7B-shaped target: prefill of all episodes in one call and
    verification of all trees in one call, both tensor-bound; times and algorithmic TFLOP/s
    (2 x 6.607e9 flop per row; the two-limb arithmetic does twice that)."""
    import torch
    from paper_2507_22424_b200.binding import SpecVLA
    from synth_inputs import configs as C, data
    torch.cuda.set_device(0)
    desc = C.OPENVLA_7B
    weights = data.make_weights(desc, C.C4.seed, device="cuda", with_draft=False)
    pre = [data.make_prefix(C.C4, episode=e, device="cuda", prefix_seed=C.C4.extra["prefix_seed"])
           for e in range(n_ep)]
    lens = [len(i) for _, i in pre]
    emb = torch.cat([e for e, _ in pre])
    ids = torch.cat([i for _, i in pre]).tolist()
    eps = list(range(n_ep))
    gpu = SpecVLA(desc, weights, max_seq=512, max_episodes=n_ep, max_rows=n_ep * 320, action_only=True)
    ms_p, ms_v = [], []
    for i in range(warmup + steps):
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record()
        first = gpu.prefill(eps, emb, ids, lens)
        b.record()
        trees = []
        for e in eps:
            tok, par, dep = data.random_tree(27, desc, seed=50 + e, max_depth=5, root_token=first[e])
            trees.append(dict(tokens=tok, parent=par, depth=dep))
        torch.cuda.synchronize()
        b2 = torch.cuda.Event(enable_timing=True)
        b2.record()
        gpu.verify_tree(eps, trees, C.C4.extra["r"])
        c.record()
        torch.cuda.synchronize()
        if i >= warmup:
            ms_p.append(a.elapsed_time(b))
            ms_v.append(b2.elapsed_time(c))
    mp, mv = statistics.median(ms_p), statistics.median(ms_v)
    rows_p, rows_v = sum(lens), 27 * n_ep
    peaks = load_peaks()
    print(json.dumps(dict(micro="batch", episodes=n_ep, prefix_rows=rows_p, tree_rows=rows_v, steps=steps,
                          prefill_ms=mp, verify_ms=mv,
                          prefill_tflops=2 * 6.607e9 * rows_p / mp / 1e9,
                          verify_tflops=2 * 6.607e9 * rows_v / mv / 1e9,
                          bf16_peak_tflops=peaks.get("bf16_tflops"), peak_source=peaks["source"],
                          note="algorithmic flops (one bf16 pass); the kernels run two limbs, i.e. twice these")),
          flush=True)
    gpu.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--micro", default=None, help="gemm:T:N:K[:M], verify:L[:T] or batch[:E] - small cases for kernel timing / ncu (see run_micro)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.micro:
        run_micro(args.micro, args.steps, args.warmup)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        import torch
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the CUDA path has no CPU fallback")
        torch.set_grad_enabled(False)
        run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
