#!/usr/bin/env python
"""Benchmark of the retrieval hot path on one B200 (replicas only at N > 1: the path does not shard).

A step = append one frame (step 1: page + pool) and answer one question (steps 2-5: retrieve, gather,
attend over all layers) on the 7B-shape, HBM-resident, 1800-frame synthetic stream.  The headline
value is the per-question retrieve+gather+attend latency; the append time is reported beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle, as it stands, on the host
cores on a bounded sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# The headline workload is BASELINE configs[1] (Qwen2-7B-like decoder, 1-hour stream at 0.5 fps, whole
# cache in HBM).  The other full-size configurations can be timed with --workload; they are parity-test
# cases, not the bench line.
WORKLOADS = {
    "7b_hbm_1800f": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=32, seed=2503, off_scale=0.5,
                         tail=0, nQ=1, appends_per_step=1),
    "7b_offload_10800f": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=10800, W=8, k=64, Nq=32, seed=2503,
                              off_scale=0.5, tail=64, nQ=1, appends_per_step=1),
    "7b_stream_batch16": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=32, Nq=(24, 64), seed=2503,
                              off_scale=0.5, tail=0, nQ=16, appends_per_step=10),
    # decode-shaped question (one token): the HBM-bound end of Eq. 3
    "7b_hbm_decode_1tok": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=1, seed=2503, off_scale=0.5,
                               tail=0, nQ=1, appends_per_step=1),
    # a short question (10 tokens = 70 rows per KV head): one row tile per unit, run as two half-streams
    "7b_hbm_short_q10": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=10, seed=2503, off_scale=0.5,
                             tail=0, nQ=1, appends_per_step=1),
    # block retrieval (Eq. 2 paragraph, b = 8): 8 blocks of 8 consecutive frames instead of 64 frames
    "7b_hbm_block8": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=32, seed=2503, off_scale=0.5,
                          tail=0, nQ=1, appends_per_step=1, b=8),
    "7b_offload_10800f_block8": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=10800, W=8, k=64, Nq=32, seed=2503,
                                     off_scale=0.5, tail=64, nQ=1, appends_per_step=1, b=8),
    # Eq. 3 in full: the question's own K/V (causal) after the retrieved context, rotary embedding with the
    # retrieved tokens at consecutive positions (base 1e6, the paper's Qwen2-based models)
    "7b_hbm_full_eq3_rope": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=32, seed=2503,
                                 off_scale=0.5, tail=0, nQ=1, appends_per_step=1, full=True, rope_theta=1e6),
    # the same with the paragraph's static variant: all context tokens at one position, no rotated copies of the keys
    "7b_hbm_full_eq3_rope_static": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=32, seed=2503,
                                        off_scale=0.5, tail=0, nQ=1, appends_per_step=1, full=True, rope_theta=1e6,
                                        rope_static=True),
    # Eq. 1, one step of stream encoding: the incoming frame's tokens attend the local window (the last W stored
    # frames, nothing retrieved) and themselves causally, then the frame's K/V are appended
    "7b_encode_frame_w8": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=0, Nq=196, seed=2503,
                               off_scale=0.5, tail=0, nQ=1, appends_per_step=1, full=True, rope_theta=1e6),
    # external retrieval (the paper's baseline retriever): SigLIP-sized frame embeddings, one selection for all layers
    "7b_hbm_external_1152": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=1800, W=8, k=64, Nq=32, seed=2503,
                                 off_scale=0.5, tail=0, nQ=1, appends_per_step=1, ext_dim=1152, tau=0.07),
    "72b_offload_1800f": dict(L=80, Hq=64, Hkv=8, D=128, Nf=196, T=1800, W=8, k=32, Nq=64, seed=2503,
                              off_scale=0.5, tail=32, nQ=1, appends_per_step=1),
    # the two offloaded configurations with the quantised host tier (FP8 E4M3 rows + scales cross the link)
    "7b_offload_10800f_fp8": dict(L=28, Hq=28, Hkv=4, D=128, Nf=196, T=10800, W=8, k=64, Nq=32, seed=2503,
                                  off_scale=0.5, tail=64, nQ=1, appends_per_step=1, host_fp8=True),
    "72b_offload_1800f_fp8": dict(L=80, Hq=64, Hkv=8, D=128, Nf=196, T=1800, W=8, k=32, Nq=64, seed=2503,
                                  off_scale=0.5, tail=32, nQ=1, appends_per_step=1, host_fp8=True),
}
WORKLOAD = dict(WORKLOADS["7b_hbm_1800f"], name="7b_hbm_1800f")
N_ROTATE = 8  # distinct questions rotated through the timed steps


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs.

    nvidia-smi needs a moment to start, so it is launched before the warm-up; mark_begin()/mark_end()
    delimit the samples that fall inside the timed region (if the region is shorter than one sampling
    period, the sample taken right after it is used)."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.begin = self.end = 0

    def _lines(self):
        return [r for r in open(self.f.name).read().splitlines() if r.strip()]

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def wait_first_sample(self):
        """Called before the barrier that opens the timed region, so that nothing here keeps the device idle
        between that barrier and the first timed step."""
        if self.p is None:
            return
        t0 = time.time()
        while not self._lines() and time.time() - t0 < 3.0:
            time.sleep(0.02)

    def mark_begin(self):
        if self.p is None:
            return
        self.begin = len(self._lines())

    def mark_end(self):
        if self.p is None:
            return
        time.sleep(0.06)  # let the sample that covers the end of the region land
        self.end = len(self._lines())

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        rows = [r.split(",") for r in self._lines()]
        os.unlink(self.f.name)
        rows = rows[max(self.begin - 1, 0):max(self.end, self.begin + 1)]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
                for n, v in zip(names, r[5:9]):
                    if v.strip().lower() == "active":
                        reasons.add(n)
            except Exception:
                continue
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch from the committed ncu capture
# (profiles/), scaled to the full workload by the layers processed; None where no capture exists.
TRAFFIC_NCU = {"7b_hbm_1800f": 848.2e6, "7b_hbm_decode_1tok": 825.0e6}


def algorithmic_bytes(w, sum_nq=None, nQ=1):
    """Bytes the method must move per question batch (all layers): representatives once, Q in / O out,
    every question's k retrieved frames' K and V once, the W window frames once."""
    sum_nq = w["Nq"] if sum_nq is None else sum_nq
    page = w["Hkv"] * 2 * w["Nf"] * w["D"] * 2
    reps = w["L"] * w["T"] * w["Hkv"] * w["D"] * 4
    if w.get("ext_dim"):  # external retrieval reads the embedding table once, for all layers
        reps = w["T"] * w["ext_dim"] * 4
    qo = 2 * w["L"] * sum_nq * w["Hq"] * w["D"] * 2
    kv = w["L"] * (nQ * w["k"] + w["W"]) * page
    kv_read = w["L"] * nQ * (w["k"] + w["W"]) * page  # what the attention kernel is asked to read
    return dict(reps=reps, q_out=qo, kv=kv, total=reps + qo + kv, attend_kernel=kv_read + qo)


def attention_flops(w, sum_nq=None):
    sum_nq = w["Nq"] if sum_nq is None else sum_nq
    return 4.0 * w["L"] * sum_nq * w["Hq"] * (w["k"] + w["W"]) * w["Nf"] * w["D"]


# ------------------------------------------------------------------------------------------ CPU oracle arm
class OracleArm:
    """The CPU oracle, as it stands, on the first `n_layers` layers of the workload.

    Set-up (untimed) computes those layers' representatives (step 1) for the whole stream.  run() times
    steps 2-5 of one question; the frames it selects are regenerated from the seeded generator instead
    of holding the 20 GB cache (input generation, excluded from the timing)."""

    def __init__(self, w, n_layers):
        from oracle import rekv_oracle as orc
        from paper_2503_00540_b200 import synth
        self.w, self.Ls, self.orc, self.synth = w, n_layers, orc, synth
        self.cores = len(os.sched_getaffinity(0))
        self.reps = torch.empty(n_layers, w["T"], w["Hkv"] * w["D"], dtype=torch.float32)
        for f in range(w["T"]):
            kf = synth.frame(w["seed"], synth.K, f, n_layers, w["Nf"], w["Hkv"], w["D"], w["off_scale"])
            for l in range(n_layers):
                self.reps[l, f] = orc.pool_frame(kf[l])

    def run(self, question_id=0):
        w, orc, synth = self.w, self.orc, self.synth
        q = synth.question(w["seed"], question_id, self.Ls, w["Nq"], w["Hq"], w["D"])
        t0 = time.perf_counter()
        t_gen = 0.0
        for l in range(self.Ls):
            s = orc.score(q[l].contiguous(), self.reps[l].contiguous(), w["Hkv"])
            idx, k_eff, _ = orc.select(s, w["T"], w["W"], w["k"])
            t1 = time.perf_counter()
            frames = idx[:k_eff].tolist() + list(range(w["T"] - w["W"], w["T"]))
            ck = torch.stack([synth.frame(w["seed"], synth.K, f, 1, w["Nf"], w["Hkv"], w["D"], w["off_scale"],
                                          layer0=l)[0] for f in frames]).contiguous()
            cv = torch.stack([synth.frame(w["seed"], synth.V, f, 1, w["Nf"], w["Hkv"], w["D"], w["off_scale"],
                                          layer0=l)[0] for f in frames]).contiguous()
            t_gen += time.perf_counter() - t1
            sub_idx = torch.arange(k_eff, dtype=torch.int32)
            kc = orc.gather(ck, sub_idx, k_eff, len(frames), w["W"])
            vc = orc.gather(cv, sub_idx, k_eff, len(frames), w["W"])
            orc.attend(q[l].contiguous(), kc, vc)
        dt = time.perf_counter() - t0 - t_gen
        return dt, dt * w["L"] / self.Ls


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if w.get("full") or w.get("ext_dim"):
        raise SystemExit("the CPU-oracle arm times steps 2-5 of the retrieval path; use a workload without full=True")
    Ls = 2
    arm = OracleArm(w, Ls)
    times = []
    for i in range(args.warmup + args.steps):
        dt, scaled = arm.run(i % N_ROTATE)
        if i >= args.warmup:
            times.append(scaled)
    cores = arm.cores
    val = sum(times) / len(times) * 1e6
    line = {
        "impl": "reference", "metric": "question_latency_us", "value": val, "unit": "us", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": val / 1e3, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        # the same keys as the CUDA arm's config (the workload is the same; what a CPU run has no use for says so)
        "config": {"workload": w["name"], "layers": w["L"], "q_heads": w["Hq"], "kv_heads": w["Hkv"],
                   "frames": w["T"], "tokens_per_frame": w["Nf"], "questions_per_batch": w["nQ"],
                   "q_tokens": w["Nq"], "top_k": w["k"], "window": w["W"], "hbm_tail_frames": w["tail"],
                   "cache_gb": 2 * w["L"] * w["T"] * w["Nf"] * w["Hkv"] * w["D"] * 2 / 1e9,
                   "l2": "not applicable: CPU oracle, inputs regenerated from the seed",
                   "parallelism": "host cores (OpenMP)",
                   "step": f"1 question (retrieve, gather, attend) on {Ls} of {w['L']} layers, scaled to all layers"},
        "cpu_baseline": {"value": val, "unit": "us", "cores": cores, "kind": "oracle",
                         "sample": f"steps 2-5 of one question on {Ls} of {w['L']} layers per step, "
                                   f"scaled x{w['L'] // Ls}"},
        "e2e": {"value": val, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ CUDA arm
def max_over_ranks(values, device, world):
    """Every reported time is the maximum over the ranks (replicas run independently)."""
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def pinned_h2d_gbs(dev, n_bytes=1 << 30, reps=5):
    """Measured pinned host -> device copy bandwidth (the host-link peak of this machine)."""
    h = torch.empty(n_bytes, dtype=torch.uint8).pin_memory()
    d = torch.empty(n_bytes, dtype=torch.uint8, device=dev)
    best = 1e30
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        d.copy_(h, non_blocking=True)
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    del h, d
    return n_bytes / best / 1e6


def run_cuda(args, w):
    import torch.distributed as dist
    from paper_2503_00540_b200 import rekv, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    K, Wu = args.steps, args.warmup
    aps, nQ = w["appends_per_step"], w["nQ"]
    n_total_steps = 2 * (K + Wu) + 4
    n_new = n_total_steps * aps
    T0 = w["T"] - n_new  # the stream ends at ~T frames after all appends
    if isinstance(w["Nq"], tuple):
        lengths = synth.question_lengths(w["seed"], nQ, w["Nq"][0], w["Nq"][1])
    else:
        lengths = [w["Nq"]] * nQ
    cu = [0]
    for n in lengths:
        cu.append(cu[-1] + n)
    w["Nq_total"] = cu[-1]

    g = rekv.ReKV(w["L"], w["Hq"], w["Hkv"], w["D"], w["Nf"], w["T"] + 8, w["W"], hbm_tail_frames=w["tail"],
                  max_q_tokens=cu[-1], max_topk=w["k"], max_questions=nQ, device=local,
                  flags=(rekv.FLAG_HOST_FP8 if w.get("host_fp8") else 0) | (rekv.FLAG_ROPE_STATIC if w.get("rope_static") else 0),
                  max_self_tokens=cu[-1] if w.get("full") else 0, rope_theta=w.get("rope_theta", 0.0),
                  ext_embed_dim=w.get("ext_dim", 0), block_frames=w.get("b", 1))
    kf = torch.empty((w["L"], w["Nf"], w["Hkv"], w["D"]), dtype=torch.bfloat16, device=dev)
    vf = torch.empty_like(kf)
    for f in range(T0):
        synth.frame(w["seed"], synth.K, f, w["L"], w["Nf"], w["Hkv"], w["D"], w["off_scale"], device=dev, out=kf)
        synth.frame(w["seed"], synth.V, f, w["L"], w["Nf"], w["Hkv"], w["D"], w["off_scale"], device=dev, out=vf)
        g.append_frame(kf, vf)
    # the frames appended inside the timed steps (a ring of 16, content irrelevant to the timing) and the
    # rotating question batches, resident in HBM
    ring_n = min(16, n_new)
    new_k = [synth.frame(w["seed"], synth.K, T0 + i, w["L"], w["Nf"], w["Hkv"], w["D"], w["off_scale"], device=dev)
             for i in range(ring_n)]
    new_v = [synth.frame(w["seed"], synth.V, T0 + i, w["L"], w["Nf"], w["Hkv"], w["D"], w["off_scale"], device=dev)
             for i in range(ring_n)]
    qs = [torch.cat([synth.question(w["seed"], r * nQ + i, w["L"], n, w["Hq"], w["D"], device=dev)
                     for i, n in enumerate(lengths)], dim=1).contiguous() for r in range(N_ROTATE)]
    out = torch.empty_like(qs[0])
    if w.get("full"):  # the questions' own K/V (N_s = N_q: the question itself), same lengths as the queries
        ks_self = torch.cat([synth.frame(w["seed"], synth.K, 1_000_000 + i, w["L"], n, w["Hkv"], w["D"], 0.0, device=dev)
                             for i, n in enumerate(lengths)], dim=1).contiguous()
        vs_self = torch.cat([synth.frame(w["seed"], synth.V, 1_000_000 + i, w["L"], n, w["Hkv"], w["D"], 0.0, device=dev)
                             for i, n in enumerate(lengths)], dim=1).contiguous()

        no_idx = torch.empty((w["L"], nQ, 0), dtype=torch.int32, device=dev)

        def ask(qt, n_vis, out):
            idx = g.retrieve(qt, cu, w["k"], n_vis)[0] if w["k"] > 0 else no_idx
            g.gather(idx, nQ, w["k"], n_vis)
            return g.attend_full(qt, ks_self, vs_self, cu, cu, out=out)
    elif w.get("ext_dim"):
        # seeded stand-ins for the external encoder's embeddings (its weights are not in this repository)
        gen = torch.Generator().manual_seed(w["seed"])
        common = torch.randn(w["ext_dim"], generator=gen)
        ext_frames = (torch.randn(w["T"] + 8, w["ext_dim"], generator=gen) + 0.7 * common).to(dev)
        ext_q = [(torch.randn(nQ, w["ext_dim"], generator=gen) + 0.7 * common).to(dev) for _ in range(N_ROTATE)]
        for f in range(T0):
            g.set_frame_embedding(f, ext_frames[f])
        ext_state = {"i": 0}

        def ask(qt, n_vis, out):
            ext_state["i"] += 1
            idx, _, _ = g.retrieve_external(ext_q[ext_state["i"] % N_ROTATE], w["k"], n_vis, w["tau"])
            g.gather(idx, nQ, w["k"], n_vis)
            return g.attend(qt, cu, out)
    else:
        def ask(qt, n_vis, out):
            return g.question(qt, cu, w["k"], n_vis, out=out)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream(dev)
    state = {"next": 0}

    def appends(src_k, src_v):
        nf = 0
        for _ in range(aps):
            j = state["next"]
            state["next"] += 1
            nf = g.append_frame(src_k[j % len(src_k)], src_v[j % len(src_v)])
            if w.get("ext_dim"):
                g.set_frame_embedding(nf, ext_frames[nf])
        return nf

    def step_device(i, ev=None):
        if ev:
            ev[0].record(stream)
        nf = appends(new_k, new_v)
        if ev:
            ev[1].record(stream)
        ask(qs[i % N_ROTATE], nf + 1, out)
        if ev:
            ev[2].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    sampler = ClockSampler(local)
    sampler.start()
    for i in range(Wu):
        step_device(i)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    sampler.wait_first_sample()
    l0 = g.launch_count()
    barrier()
    sampler.mark_begin()
    t_begin.record(stream)
    for i in range(K):
        step_device(i, evs[i])
    t_end.record(stream)
    barrier()
    sampler.mark_end()
    launches = g.launch_count() - l0
    clocks = sampler.stop()
    total_ms = t_begin.elapsed_time(t_end)
    q_us = [e[1].elapsed_time(e[2]) * 1e3 / nQ for e in evs]
    a_us = [e[0].elapsed_time(e[1]) * 1e3 / aps for e in evs]
    g.check_status()

    # attention-kernel duration (library-internal events on the launching stream) and bytes over the host link
    # (the event records stand between the attention kernel and its neighbours, so they are on only here)
    att_us, link_bytes = [], 0
    stage_us = {"retrieve": [], "pull": [], "merge": []}
    g.set_timing(True)
    for i in range(min(K, 8)):
        ask(qs[i % N_ROTATE], g.stats().frames, out)
        torch.cuda.synchronize()
        st = g.stats()
        att_us.append(st.last_attend_kernel_us)
        stage_us["retrieve"].append(st.last_retrieve_us)
        stage_us["pull"].append(st.last_pull_us)
        stage_us["merge"].append(st.last_merge_us)
        link_bytes = st.last_link_bytes
    g.set_timing(False)

    # ---- end to end: inputs in pinned host memory, result read back, every step ----
    hk = [t.cpu().pin_memory() for t in new_k[:2]]
    hv = [t.cpu().pin_memory() for t in new_v[:2]]
    hq = [t.cpu().pin_memory() for t in qs]
    hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    dq = torch.empty_like(qs[0])

    # The headline metric is the question's latency, so `e2e` is the question end to end: its queries copied from
    # pinned host memory, steps 2-5, the output copied back (ev[1] .. ev[2]); the bytes declared for it are the
    # bytes copied inside that region.  The whole step -- the frame's K/V copied from pinned host memory and
    # appended first (ev[0] .. ev[2]) -- is reported beside it with its own byte count.
    def step_e2e(i, ev=None):
        nf = 0
        if ev:
            ev[0].record(stream)
        for a in range(aps):
            state["next"] += 1
            kf.copy_(hk[(i + a) % 2], non_blocking=True)
            vf.copy_(hv[(i + a) % 2], non_blocking=True)
            nf = g.append_frame(kf, vf)
            if w.get("ext_dim"):
                g.set_frame_embedding(nf, ext_frames[nf])
        if ev:
            ev[1].record(stream)
        dq.copy_(hq[i % N_ROTATE], non_blocking=True)
        ask(dq, nf + 1, out)
        hout.copy_(out, non_blocking=True)
        if ev:
            ev[2].record(stream)

    for i in range(Wu):
        step_e2e(i)
    evs2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    barrier()
    for i in range(K):
        step_e2e(i, evs2[i])
    barrier()
    e2e_us = [e[1].elapsed_time(e[2]) * 1e3 / nQ for e in evs2]
    e2e_step_us = [e[0].elapsed_time(e[2]) * 1e3 for e in evs2]
    g.check_status()

    def mean(x):
        return sum(x) / len(x)

    # steps 2-3 alone (question vectors, scores, selection): frames scored per second
    n_vis = g.stats().frames
    ev_r = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    if w.get("ext_dim"):
        def retrieve_only(i):
            g.retrieve_external(ext_q[i % N_ROTATE], w["k"], n_vis, w["tau"])
    else:
        def retrieve_only(i):
            g.retrieve(qs[i % N_ROTATE], cu, w["k"], n_vis)
    for i in range(3):
        retrieve_only(i)
    torch.cuda.synchronize()
    ev_r[0].record(stream)
    for i in range(10):
        retrieve_only(i)
    ev_r[1].record(stream)
    torch.cuda.synchronize()
    retrieve_us = ev_r[0].elapsed_time(ev_r[1]) * 1e3 / 10

    # layer-sequential mode: one call per layer, as a decoder that makes layer l+1's queries from layer
    # l's output drives the path; HBM-resident caches replay one captured CUDA graph per layer (no host
    # work between layers), offloaded caches issue the calls eagerly (their side stream is not capturable)
    q_l = qs[0].clone()
    layer_calls = []
    if w.get("full"):  # Eq. 3 in full, layer by layer: the decoder layer's call with its own Q, K, V (eager calls)
        for l in range(w["L"]):
            layer_calls.append(lambda l=l: g.question_layer_full(l, q_l[l], ks_self[l], vs_self[l], cu, cu, w["k"],
                                                                 n_vis, out=out[l]))
    elif w["tail"] == 0:
        cap = torch.cuda.Stream(dev)
        cap.wait_stream(stream)
        with torch.cuda.stream(cap):
            for l in range(w["L"]):
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=cap):
                    g.question_layer(l, q_l[l], cu, w["k"], n_vis, out=out[l])
                layer_calls.append(gr.replay)
            # the same 28 calls as consecutive nodes of ONE graph: what a decoder captured whole (its own
            # kernels between the layers) pays for the path, without a graph launch per layer
            gr_all = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr_all, stream=cap):  # (used below for workloads without Eq. 3 in full)
                for l in range(w["L"]):
                    g.question_layer(l, q_l[l], cu, w["k"], n_vis, out=out[l])
        stream.wait_stream(cap)
    else:
        for l in range(w["L"]):
            layer_calls.append(lambda l=l: g.question_layer(l, q_l[l], cu, w["k"], n_vis, out=out[l]))
    n_seq = 3 if w["tail"] else 10
    for i in range(2 + n_seq):
        if i == 2:
            torch.cuda.synchronize()
            ev_r[0].record(stream)
        q_l.copy_(qs[i % N_ROTATE])
        for call in layer_calls:
            call()
    ev_r[1].record(stream)
    torch.cuda.synchronize()
    layer_seq_us = ev_r[0].elapsed_time(ev_r[1]) * 1e3 / n_seq / nQ
    layer_seq_one_graph_us = None
    decode_layers_us = None
    if w["tail"] == 0 and not w.get("full") and max(lengths) * (w["Hq"] // w["Hkv"]) > 16:
        # generation after the question: every new token attends the same retrieved context, layer by layer
        # (rekv_attend_layer, one query row per question), all layers of a token as consecutive nodes of one graph
        cu1 = list(range(nQ + 1))
        qd = [synth.question(w["seed"], 900 + r, w["L"], nQ, w["Hq"], w["D"], device=dev) for r in range(2)]
        qd_buf, od_buf = qd[0].clone(), torch.empty_like(qd[0])
        g.question(qs[0], cu, w["k"], n_vis, out=out)            # the context the tokens reuse
        g.gather(g.retrieve(qs[0], cu, w["k"], n_vis)[0], nQ, w["k"], n_vis)
        cap2 = torch.cuda.Stream(dev)
        cap2.wait_stream(stream)
        with torch.cuda.stream(cap2):
            gr_dec = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr_dec, stream=cap2):
                for l in range(w["L"]):
                    g.attend_layer(l, qd_buf[l], cu1, out=od_buf[l])
        stream.wait_stream(cap2)
        for i in range(2 + 20):
            if i == 2:
                torch.cuda.synchronize()
                ev_r[0].record(stream)
            qd_buf.copy_(qd[i % 2])
            gr_dec.replay()
        ev_r[1].record(stream)
        torch.cuda.synchronize()
        decode_layers_us = ev_r[0].elapsed_time(ev_r[1]) * 1e3 / 20
    if w["tail"] == 0 and not w.get("full"):
        for i in range(2 + n_seq):
            if i == 2:
                torch.cuda.synchronize()
                ev_r[0].record(stream)
            q_l.copy_(qs[i % N_ROTATE])
            gr_all.replay()
        ev_r[1].record(stream)
        torch.cuda.synchronize()
        layer_seq_one_graph_us = ev_r[0].elapsed_time(ev_r[1]) * 1e3 / n_seq / nQ
    g.check_status()

    q_sorted = sorted(q_us)
    q_lat, ms_step, e2e_lat, app_us, att_kernel_us, retrieve_us, layer_seq_us, q_median, q_min, e2e_step = max_over_ranks(
        [mean(q_us), total_ms / K, mean(e2e_us), mean(a_us), mean(att_us), retrieve_us, layer_seq_us,
         q_sorted[len(q_sorted) // 2], q_sorted[0], mean(e2e_step_us)], dev, world)

    if rank == 0:
        peaks = measured_peaks()
        ab = algorithmic_bytes(w, cu[-1], nQ)
        fl = attention_flops(w, cu[-1])
        line = {
            "metric": "question_latency_us", "value": q_lat, "unit": "us", "n_gpus": world, "steps": K, "warmup": Wu,
            "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w["name"], "layers": w["L"], "q_heads": w["Hq"], "kv_heads": w["Hkv"],
                       "frames": w["T"], "tokens_per_frame": w["Nf"], "questions_per_batch": nQ,
                       "q_tokens": lengths if nQ > 1 else lengths[0], "top_k": w["k"], "window": w["W"],
                       "hbm_tail_frames": w["tail"],
                       "cache_gb": 2 * w["L"] * w["T"] * w["Nf"] * w["Hkv"] * w["D"] * 2 / 1e9,
                       "l2": f"inputs larger than L2: a question batch streams {ab['total'] / 1e9:.2f} GB, "
                             f"{N_ROTATE} batches rotate",
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "step": f"append {aps} frame(s) + {nQ} question(s) (retrieve, gather, attend; all layers)"},
            "question": {"bytes_per_batch": ab["total"], "gbs": ab["total"] / (q_lat * nQ * 1e-6) / 1e9,
                         "hbm_frac": ab["total"] / (q_lat * nQ * 1e-6) / 1e9 / peaks["hbm_gbs"],
                         "attention_tflops": fl / (q_lat * nQ * 1e-6) / 1e12,
                         "median_us": q_median, "min_us": q_min, "per_step_us": [round(x, 1) for x in q_us],
                         "layer_sequential_us": layer_seq_us,
                         "layer_sequential_one_graph_us": layer_seq_one_graph_us,
                         "decode_token_layer_by_layer_us": decode_layers_us,
                         "layer_sequential_mode": ("one eager rekv_question_layer_full call per layer" if w.get("full")
                                                   else "one CUDA graph replay per layer" if w["tail"] == 0
                                                   else "one eager call per layer"),
                         "retrieve_us_per_batch": retrieve_us,
                         "frames_scored_per_s_all_gpus": (world * (1 if w.get("ext_dim") else w["L"]) * n_vis * nQ
                                                          / (retrieve_us * 1e-6)),
                         "questions_per_s_all_gpus": world * 1e6 / q_lat},
            "append_us": app_us,
            # the library's own stage timings of a question (rekv_stats with the event records on; each record stands
            # between two kernels, so the stages add up to a little more than the untimed question)
            "stages_us": {k: (sum(v) / len(v) if v else None) for k, v in stage_us.items()},
            "e2e": {"value": e2e_lat, "unit": "us",
                    "h2d_bytes_per_step": dq.numel() * 2,
                    "d2h_bytes_per_step": out.numel() * 2,
                    "region": "per question: queries H2D from pinned memory, steps 2-5, output D2H",
                    "whole_step_us": e2e_step,
                    "whole_step_h2d_bytes": aps * 2 * kf.numel() * 2 + dq.numel() * 2,
                    "whole_step_region": f"{aps} frame(s) K/V H2D + append, then the question batch as above"},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if w["tail"] == 0:
            achieved = ab["attend_kernel"] / (att_kernel_us * 1e-6) / 1e9
            line["roofline"] = {"kernel": ("attend_decode_kernel (step 5)" if max(lengths) * (w["Hq"] // w["Hkv"]) <= 16
                                           else "attend_tc5_kernel (step 5)"), "bound": "hbm", "achieved": achieved,
                                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                                "traffic": TRAFFIC_NCU.get(w["name"]), "peak_source": peaks["source"],
                                "kernel_us": att_kernel_us,
                                "tensor_tflops": fl / (att_kernel_us * 1e-6) / 1e12,
                                "tensor_frac": fl / (att_kernel_us * 1e-6) / 1e12 / peaks["bf16_tflops"],
                                "covers": ("the whole of step 5: when no merge launch follows (stages_us.merge = 0) the "
                                           "kernel also joins the units cut between CTAs, which are not among the "
                                           "algorithmic bytes")}
        else:
            link = pinned_h2d_gbs(dev)
            achieved = link_bytes / (q_lat * 1e-6) / 1e9
            line["roofline"] = {"kernel": "page_table_pull_kernel (step 4, host tier)", "bound": "host_link",
                                "achieved": achieved, "peak": link, "unit": "GB/s", "frac": achieved / link,
                                "traffic": None, "peak_source": "pinned H2D copy measured in this run",
                                "link_bytes_per_question": link_bytes}
        if not args.no_cpu_baseline and world == 1 and w["name"] == "7b_hbm_1800f":
            arm = OracleArm(w, w["L"])
            runs = [arm.run(i) for i in range(3)]  # three different questions, about 11 s of CPU work
            dt = sum(r[0] for r in runs)
            scaled = sum(r[1] for r in runs) / len(runs)
            line["cpu_baseline"] = {"value": scaled * 1e6, "unit": "us", "cores": arm.cores, "kind": "oracle",
                                    "sample": f"steps 2-5 of three whole questions, all {w['L']} layers, mean "
                                              f"({dt:.1f} s of CPU work; pooling and input generation untimed)"}
        print(json.dumps(line))
    g.close()
    if world > 1:
        dist.destroy_process_group()


def rank_plumbing_check(args):
    """Only the rank plumbing of the replicas-only N > 1 run, on CPU with the gloo backend: rendezvous from the
    launcher's environment, barrier, maximum over the ranks of a per-rank time.  Rank 0 prints one JSON line.
    The CPU tests use it to run the `--gpus N` launcher without a GPU."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    worst = max_over_ranks([100.0 + rank, 5.0 - rank], torch.device("cpu"), world)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"plumbing_check": True, "n_gpus": world, "max_over_ranks": worst}))


def launch_replicas(args):
    """`--gpus N` without a launcher's environment: start the N replica processes here, one per device, the way
    the N > 1 run is specified (torch.distributed.run on one node, rendezvous on 127.0.0.1).  The replicas are
    independent; the process group only carries the barriers and the maximum over the ranks."""
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")            # the communicator's set-up lines, kept off stdout
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="7b_hbm_1800f", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=None, help="profiling only: fewer layers than the workload")
    ap.add_argument("--frames", type=int, default=None, help="profiling only: a shorter stream")
    ap.add_argument("--plumbing-check", action="store_true",
                    help="run only the rank plumbing (gloo, CPU): what the CPU tests use to exercise --gpus N")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "cuda" or args.plumbing_check):
        sys.exit(launch_replicas(args))
    if args.plumbing_check:
        return rank_plumbing_check(args)
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    w = dict(WORKLOADS[args.workload], name=args.workload)
    if args.layers or args.frames:
        w["L"] = args.layers or w["L"]
        w["T"] = args.frames or w["T"]
        w["name"] = f"{w['name']}_reduced_L{w['L']}_T{w['T']}_for_profiling"
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
