"""Benchmark of the verify step (attention + accept/resample + gamma update).

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload c5]

One step = one pass of the whole hot path over one batch of seeded synthetic
input.  The default workload is the largest configuration (Llama-3.1-70B-shaped:
batch 128, 64q/8kv heads, ragged contexts 512..16384, V = 128256, gamma = 16 for
every sequence, temperature 1, noise sigma 1).  The controller state is reset to
the same values before every step (one small device-to-device copy inside the
timed region), so that every timed step does the same work on the same inputs.

N > 1: one process per GPU (under torchrun, or started by this script when it is
run without a launcher); sequences are independent, so there is no data-path
collective: every rank runs its own batch (--scaling weak, the default) or its
share of one batch cut by cached tokens (--scaling strong); value = all ranks'
tokens / max time.

--impl reference times the float64 CPU oracle on a bounded sample of the same
workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2504_00030_b200 import shard, synth  # noqa: E402

METRIC = "verified tokens/sec (verify step: attention + accept/resample + gamma update)"
UNIT = "tokens/s"
GT = dict(eta=0.5, delta=2.0, gamma_min=1)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def workload_inputs(cfg, rank, batch=None, gamma=None, gamma_max=None):
    cfg = synth.scaled(cfg, seed=shard.rank_seed(cfg.seed, rank))
    if gamma_max is not None:
        cfg = synth.scaled(cfg, gamma_max=gamma_max)
    if gamma is not None:
        cfg = synth.scaled(cfg, gamma_lo=gamma, gamma_hi=gamma)
    if batch:
        cfg = synth.scaled(cfg, batch=batch)
    seq_len, gamma = synth.draw_lengths(cfg)
    cu_q, cu_d = synth.padded_offsets(cfg.batch, cfg.gamma_max)
    return cfg, seq_len, gamma, cu_q, cu_d


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_step(cfg, seq_len, gamma, cu_q, cu_d, kv, q, li, n_seq):
    """The oracle, as it stands, on the first n_seq sequences of the batch; returns
    (seconds, verified tokens)."""
    import oracle
    sl, g = seq_len[:n_seq], gamma[:n_seq]
    cq, cd = cu_q[:n_seq + 1], cu_d[:n_seq + 1]
    t0 = time.perf_counter()
    oracle.verify_attn(q[:cq[-1]], kv.k_pool, kv.v_pool, kv.strides, kv.block_table[:n_seq], sl, g, cq,
                       cfg.hq, cfg.hkv, cfg.page_size, float(np.float32(cfg.head_dim ** -0.5)))
    res = oracle.accept_sample(li.target_logits[:cq[-1]], li.draft_logits[:cd[-1]], li.draft_tokens[:cd[-1]],
                               li.u_accept[:cd[-1]], li.u_sample[:n_seq], cfg.temperature, g, cq, cd,
                               cfg.gamma_max)
    oracle.gamma_tune_update(res.n_accepted, g.astype(np.float64), g, sl, GT["eta"], GT["delta"],
                             GT["gamma_min"], cfg.gamma_max, oracle.MODE_GT_PROPOSED, True)
    dt = time.perf_counter() - t0
    return dt, int((res.n_accepted + 1).sum())


def sample_inputs(cfg, seq_len, gamma, cu_q, cu_d, n_seq):
    """Inputs of the first n_seq sequences only (the oracle arm never needs the rest)."""
    sub = synth.scaled(cfg, batch=n_seq)
    kv = synth.make_kv(sub, seq_len[:n_seq])
    cq, cd = cu_q[:n_seq + 1], cu_d[:n_seq + 1]
    q = synth.make_q(sub, int(cq[-1]))
    li = synth.make_logits(sub, gamma[:n_seq], cq, cd)
    return sub, kv, q, li


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    cfg, seq_len, gamma, cu_q, cu_d = workload_inputs(synth.CONFIGS[args.workload], 0, args.batch, args.gamma, args.gamma_max)
    n_seq = min(args.oracle_seqs or 4, cfg.batch)
    sub, kv, q, li = sample_inputs(cfg, seq_len, gamma, cu_q, cu_d, n_seq)
    times, toks = [], 0
    for it in range(args.warmup + args.steps):
        dt, toks = oracle_step(sub, seq_len, gamma, cu_q, cu_d, kv, q, li, n_seq)
        if it >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = toks * len(times) / total
    sample = f"first {n_seq} of {cfg.batch} sequences of {cfg.name}, whole step per sample"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(cfg, gamma, "host memory only"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(cfg, gamma, cache_note):
    return {"workload": f"{cfg.name}: batch {cfg.batch}, {cfg.hq}q/{cfg.hkv}kv heads, head_dim {cfg.head_dim}, "
                        f"contexts {cfg.ctx_lo}-{cfg.ctx_hi}, paged KV (16) bf16, V={cfg.vocab}, "
                        f"gamma {int(gamma.min())}..{int(gamma.max())} (max {cfg.gamma_max}), "
                        f"T={cfg.temperature}, sigma={cfg.sigma_noise}",
            "global_batch": cfg.batch, "parallelism": "sequences sharded per GPU, no collective",
            "controller": f"GammaTune eta={GT['eta']} delta={GT['delta']} [{GT['gamma_min']},{cfg.gamma_max}], "
                          "state reset before each step",
            "cache": cache_note}


# ------------------------------------------------------------------------------------------ GPU arm
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out = self.proc.communicate(timeout=5)[0]
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out = self.proc.communicate()[0]
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in out.strip().splitlines():
            f = [x.strip() for x in row.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


def profiled_traffic_ratio():
    """DRAM traffic of the attention main kernel per algorithmic byte, read from the committed ncu summary
    (profiles/attn_tq_kernel_c5_batch32.md: dram__bytes_read.sum + dram__bytes_write.sum of one launch over the
    algorithmic bytes of that launch).  The summary names the kernel sources it was taken from by hash; when
    they have changed since, or the file cannot be read, there is no figure (None)."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", "attn_tq_kernel_c5_batch32.md")
    try:
        text = open(path).read()
        h = hashlib.sha256()
        for name in ATTN_KERNEL_SOURCES:
            h.update(open(os.path.join(ROOT, "paper_2504_00030_b200", "csrc", name), "rb").read())
        m_hash = re.search(r"kernel sources sha256: ([0-9a-f]{64})", text)
        m_ratio = re.search(r"traffic per algorithmic byte: ([0-9.]+)", text)
        if m_hash is None or m_ratio is None or m_hash.group(1) != h.hexdigest():
            return None
        return float(m_ratio.group(1))
    except (OSError, ValueError):
        return None


ATTN_KERNEL_SOURCES = ("attn_tq.cu", "attn_tc.cu", "attn_softmax.cuh", "attn_sched.cuh", "attn_common.cuh", "tc_ptx.cuh",
                       "common.cuh")


class VerifyStep:
    """Device-resident state of one workload and the three calls of its verify step."""

    def __init__(self, sv, torch, cfg, seq_len, gamma, cu_q, cu_d, dev, reserve, host_copies=False):
        import ctypes as C
        self.sv, self.torch, self.cfg, self.C = sv, torch, cfg, C
        self.seq_len, self.gamma, self.cu_q, self.cu_d = seq_len, gamma, cu_q, cu_d
        B, gmax = cfg.batch, cfg.gamma_max
        self.n_q, self.n_d = int(cu_q[-1]), int(cu_d[-1])
        self.kv = synth.make_kv(cfg, seq_len, reserve_tokens=reserve)
        self.q_np = synth.make_q(cfg, self.n_q)
        self.li = synth.make_logits(cfg, gamma, cu_q, cu_d)

        def up(a):
            return torch.from_numpy(np.ascontiguousarray(a)).to(dev)

        def up_bf16(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)

        self.up, self.up_bf16, self.dev = up, up_bf16, dev
        self.k_pool, self.v_pool = up_bf16(self.kv.k_pool), up_bf16(self.kv.v_pool)
        self.pool = sv.spec_kv_pool_register(self.k_pool, self.v_pool)
        self.bt = up(self.kv.block_table)
        self.max_len = int(seq_len.max()) + reserve
        li = self.li
        if host_copies:
            pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
            self.q_h = torch.from_numpy(self.q_np.view(np.int16)).view(torch.bfloat16).pin_memory()
            self.tl_h, self.dl_h = pin(li.target_logits), pin(li.draft_logits)
            self.x_h, self.ua_h, self.us_h = pin(li.draft_tokens), pin(li.u_accept), pin(li.u_sample)
            self.q = self.q_h.to(dev)
            self.tl, self.dl = self.tl_h.to(dev), self.dl_h.to(dev)
            self.x, self.ua, self.us = self.x_h.to(dev), self.ua_h.to(dev), self.us_h.to(dev)
        else:
            self.q = up_bf16(self.q_np)
            self.tl, self.dl = up(li.target_logits), up(li.draft_logits)
            self.x, self.ua, self.us = up(li.draft_tokens), up(li.u_accept), up(li.u_sample)
        self.o = torch.zeros_like(self.q)
        self.n_acc = torch.zeros(B, dtype=torch.int32, device=dev)
        self.toks = torch.zeros((B, gmax + 1), dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        # controller state in one buffer so that one copy resets it: gbar | gamma | seq_len | cu_q | cu_d
        nb = 8 * B + 4 * B + 4 * B + 4 * (B + 1) + 4 * (B + 1)
        self.state = torch.zeros(nb, dtype=torch.uint8, device=dev)
        off = 0
        self.gbar = self.state[off:off + 8 * B].view(torch.float64); off += 8 * B
        self.g = self.state[off:off + 4 * B].view(torch.int32); off += 4 * B
        self.sl = self.state[off:off + 4 * B].view(torch.int32); off += 4 * B
        self.cq = self.state[off:off + 4 * (B + 1)].view(torch.int32); off += 4 * (B + 1)
        self.cd = self.state[off:off + 4 * (B + 1)].view(torch.int32)
        self.gbar.copy_(up(gamma.astype(np.float64)))
        self.g.copy_(up(gamma)); self.sl.copy_(up(seq_len)); self.cq.copy_(up(cu_q)); self.cd.copy_(up(cu_d))
        self.state0 = self.state.clone()
        gcfg = sv.GammaConfig(GT["eta"], GT["delta"], GT["gamma_min"], gmax, sv.SV_GT_PROPOSED, True)
        self.ws_a = torch.empty(max(256, sv.spec_verify_attn_workspace_bytes(B, gmax, cfg.hq, cfg.hkv, cfg.head_dim,
                                                                             self.max_len)), dtype=torch.uint8, device=dev)
        self.ws_s = torch.empty(max(256, sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab)), dtype=torch.uint8,
                                device=dev)
        self.ap = sv.attn_params(self.q, self.o, self.pool, self.bt, self.sl, self.g, self.cq, gmax, self.max_len,
                                 device_status=self.status)
        self.sp = sv.accept_params(self.tl, self.dl, self.x, self.ua, self.us, cfg.temperature, self.g, self.cq, self.cd,
                                   gmax, self.n_acc, self.toks, device_status=self.status)
        self.gp = sv.gamma_params(self.n_acc, self.gbar, self.g, self.sl, self.cq, self.cd, gcfg, device_status=self.status)
        self.lib = sv.load()
        self.stream = torch.cuda.current_stream()
        self.sptr = C.c_void_p(self.stream.cuda_stream)

    def check(self, st, what):
        if st != 0:
            raise RuntimeError(f"{what}: {self.sv.status_str(st)}")

    def calls(self):
        C, lib = self.C, self.lib
        self.check(lib.spec_verify_attn(C.byref(self.ap), self.ws_a.data_ptr(), self.ws_a.numel(), self.sptr), "attn")
        yield
        self.check(lib.spec_accept_sample(C.byref(self.sp), self.ws_s.data_ptr(), self.ws_s.numel(), self.sptr), "accept")
        yield
        self.check(lib.gamma_tune_update(C.byref(self.gp), self.sptr), "gamma")
        yield

    def step(self, ev=None):
        """One verify step; the controller state is reset first so that every step does the same work."""
        self.state.copy_(self.state0, non_blocking=True)
        if ev is not None: ev[0].record(self.stream)
        for i, _ in enumerate(self.calls()):
            if ev is not None: ev[i + 1].record(self.stream)

    def graph_us(self, steps):
        """The step captured once into a CUDA graph and replayed `steps` times: microseconds per replay, or None
        if the capture is refused.  What a caller gains on the launch-bound small workloads."""
        torch, C = self.torch, self.C
        keep = (self.stream, self.sptr)
        side = torch.cuda.Stream()
        self.stream, self.sptr = side, C.c_void_p(side.cuda_stream)
        try:
            torch.cuda.synchronize()
            with torch.cuda.stream(side):
                self.step()
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                self.step()
            torch.cuda.synchronize()
            for _ in range(3):
                graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            return 1e3 * e0.elapsed_time(e1) / steps
        except RuntimeError:
            return None
        finally:
            self.stream, self.sptr = keep

    def evolve(self, n):
        """The controller runs n steps on its own acceptance counts (no reset); the timed steps then start from
        the state it reached: a GammaTune-driven mix of draft lengths instead of gamma_max everywhere."""
        self.state.copy_(self.state0)
        for _ in range(n):
            for _ in self.calls():
                pass
        self.torch.cuda.synchronize()
        self.state0 = self.state.clone()
        self.gamma = self.g.cpu().numpy().copy()
        self.seq_len = self.sl.cpu().numpy().copy()

    def timed(self, steps, warmup, barrier):
        """Whole-step time from one pair of events around `steps` steps enqueued back to back (nothing but the
        step's own calls and the state reset on the stream, so that each kernel can be set up while its
        predecessor drains), then the same number of steps again with an event after every call for the
        breakdown."""
        torch = self.torch
        for _ in range(warmup):
            self.step()
        barrier()
        e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = self.sv.sv_launch_count()
        barrier()
        e_begin.record(self.stream)
        for it in range(steps):
            self.step()
        e_end.record(self.stream)
        barrier()
        launches = self.sv.sv_launch_count() - launches0
        assert self.status.item() == 0, f"device status {self.status.item()}"
        tokens = int((self.n_acc + 1).sum().item())           # identical every step (same inputs, same state)
        # The breakdown pass: after a pause and a short warm-up, so that it runs in the clock state of the timed
        # pass (this GPU lowers its SM clock after about 50 ms of continuous load; the timed pass ends before that).
        time.sleep(0.5)
        for _ in range(3):
            self.step()
        barrier()
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        for it in range(steps):
            self.step(evs[it])
        barrier()
        return {"ms_total": e_begin.elapsed_time(e_end), "tokens": tokens, "launches": launches,
                "attn": float(np.mean([e[0].elapsed_time(e[1]) for e in evs])),
                "accept": float(np.mean([e[1].elapsed_time(e[2]) for e in evs])),
                "gamma": float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))}


def config_lines(sv, torch, dev, steps, peak):
    """Step times of the other workloads (c1..c4: parity-test cases with their own byte floors), one entry each."""
    out = {}
    for name in ("c1", "c2", "c3", "c4"):
        cfg, seq_len, gamma, cu_q, cu_d = workload_inputs(synth.CONFIGS[name], 0, None, None, None)
        vs = VerifyStep(sv, torch, cfg, seq_len, gamma, cu_q, cu_d, dev, 2 * (cfg.gamma_max + 1))
        r = vs.timed(steps, 5, torch.cuda.synchronize)
        attn_b, acc_b = synth.algorithmic_bytes(cfg, seq_len, gamma)
        us = 1e3 * r["ms_total"] / steps
        out[name] = {"step_us": us, "attention_us": 1e3 * r["attn"], "accept_us": 1e3 * r["accept"],
                     "gamma_update_us": 1e3 * r["gamma"], "bytes": attn_b + acc_b,
                     "frac_of_8tbs": (attn_b + acc_b) / (us * 1e-6) / 8e12,
                     "frac_of_measured": (attn_b + acc_b) / (us * 1e-6) / 1e9 / peak,
                     "verified_tokens_per_s": r["tokens"] / (us * 1e-6),
                     "graph_step_us": vs.graph_us(steps)}       # the same step as one CUDA graph launch
        del vs
        torch.cuda.empty_cache()
    return out


def strong_share(base_cfg, rank, world, batch=None, gamma=None, gamma_max=None):
    """Strong scaling: one batch for the whole job (drawn as rank 0 draws it), cut into contiguous runs of
    sequences with equal numbers of cached tokens (the attention stage's bytes); returns rank's own run as a
    workload of its own (configuration with the local batch size, rebased row offsets) and the whole batch size."""
    cfg, seq_len, g, cu_q, cu_d = workload_inputs(base_cfg, 0, batch, gamma, gamma_max)
    bounds = shard.balanced_bounds(seq_len, world)
    lb = shard.local_batch(bounds, rank, seq_len, g, cu_q, cu_d)
    if lb.count == 0:
        raise RuntimeError(f"rank {rank} got no sequences: batch {cfg.batch} over {world} ranks")
    local = synth.scaled(cfg, batch=lb.count, seed=shard.rank_seed(cfg.seed, rank))
    return local, lb.seq_len, lb.gamma, lb.cu_q, lb.cu_d, cfg.batch


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2504_00030_b200 import binding as sv

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    DEV = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(DEV))

    base_cfg = synth.CONFIGS[args.workload]
    if args.scaling == "strong" and world > 1:
        cfg, seq_len, gamma, cu_q, cu_d, global_batch = strong_share(base_cfg, rank, world, args.batch, args.gamma,
                                                                     args.gamma_max)
    else:
        cfg, seq_len, gamma, cu_q, cu_d = workload_inputs(base_cfg, rank, args.batch, args.gamma, args.gamma_max)
        global_batch = cfg.batch * world
    B, gmax = cfg.batch, cfg.gamma_max
    reserve = (2 + args.evolve) * (gmax + 1)
    vs = VerifyStep(sv, torch, cfg, seq_len, gamma, cu_q, cu_d, DEV, reserve, host_copies=True)
    lib, C, stream, sptr, check = vs.lib, vs.C, vs.stream, vs.sptr, vs.check
    state, status = vs.state, vs.status
    n_q, n_d = vs.n_q, vs.n_d

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.evolve > 0:
        vs.evolve(args.evolve)
        gamma, seq_len = vs.gamma, vs.seq_len
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    r = vs.timed(args.steps, args.warmup, barrier)
    clocks = sampler.stop() if rank == 0 else None
    ms_total, tokens, launches = r["ms_total"], r["tokens"], r["launches"]
    t_attn, t_acc, t_gam = r["attn"], r["accept"], r["gamma"]
    state0 = vs.state0

    # ---- end to end through the host-buffer entry point
    n_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    tok_h = torch.zeros((B, gmax + 1), dtype=torch.int32).pin_memory()
    g_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    o_h = torch.zeros(vs.q_h.shape, dtype=torch.bfloat16).pin_memory()
    io = sv.step_host_io(vs.q_h, vs.tl_h, vs.dl_h, vs.x_h, vs.ua_h, vs.us_h, n_q, n_d, n_h, tok_h, g_h, o_h)
    h2d = sum(t.numel() * t.element_size() for t in (vs.q_h, vs.tl_h, vs.dl_h, vs.x_h, vs.ua_h, vs.us_h))
    d2h = sum(t.numel() * t.element_size() for t in (n_h, tok_h, g_h, o_h))
    e2e_steps = max(3, min(args.steps, args.e2e_steps))

    def e2e_step():
        state.copy_(state0, non_blocking=True)
        check(lib.spec_verify_step_host(C.byref(io), C.byref(vs.ap), vs.ws_a.data_ptr(), vs.ws_a.numel(), C.byref(vs.sp),
                                        vs.ws_s.data_ptr(), vs.ws_s.numel(), C.byref(vs.gp), sptr), "step_host")
        stream.synchronize()                           # the caller reads the host results every step

    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_tokens = int((n_h + 1).sum().item())
    assert e2e_tokens == tokens

    def median_us(fn, n=10):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for _ in range(3):
            fn()
        for e_a, e_b in evs:
            e_a.record(stream)
            fn()
            e_b.record(stream)
        barrier()
        return 1e3 * float(np.median([e_a.elapsed_time(e_b) for e_a, e_b in evs]))

    # ---- GammaTune+ early stop (not part of the step above): one streaming pass over the draft rows
    n_dr = torch.zeros(B, dtype=torch.int32, device=DEV)
    ws_d = torch.empty(max(256, sv.spec_draft_stop_workspace_bytes(B, gmax, cfg.vocab)), dtype=torch.uint8,
                       device=DEV)
    dp = sv.draft_stop_params(vs.dl, cfg.temperature, 0.5, vs.g, vs.cd, gmax, n_dr, device_status=status)
    state.copy_(state0)
    t_ds = median_us(lambda: check(lib.spec_draft_stop(C.byref(dp), ws_d.data_ptr(), ws_d.numel(), sptr), "draft_stop"))
    ds_bytes = int(gamma.sum()) * cfg.vocab * 4

    # ---- one drafting step with the confidence stop (not part of the step above): a row of draft logits per
    # sequence (the first B rows of the block's draft logits), token and top probability, state advanced
    n_st = torch.zeros(B, dtype=torch.int32, device=DEV)
    act_st = torch.ones(B, dtype=torch.int32, device=DEV)
    tok_st = torch.zeros(max(int(cu_d[-1]), 1), dtype=torch.int32, device=DEV)
    ws_st = torch.empty(max(256, sv.spec_draft_step_workspace_bytes(B, cfg.vocab)), dtype=torch.uint8, device=DEV)
    stp = sv.draft_step_params(vs.dl[:B], cfg.temperature, 0.0, vs.us, vs.g, vs.cd, gmax, n_st, act_st, tok_st,
                               device_status=status)

    def draft_step_once():
        n_st.zero_()            # every call drafts position 0 of every sequence again
        act_st.fill_(1)
        check(lib.spec_draft_step(C.byref(stp), ws_st.data_ptr(), ws_st.numel(), sptr), "draft_step")
    t_st = median_us(draft_step_once)
    st_bytes = B * cfg.vocab * 4

    # ---- accept / resample with the logits stored as bf16 (not part of the step above): same call, half the bytes
    tl16, dl16 = vs.tl.to(torch.bfloat16), vs.dl.to(torch.bfloat16)
    n16 = torch.zeros(B, dtype=torch.int32, device=DEV)
    tok16 = torch.zeros((B, gmax + 1), dtype=torch.int32, device=DEV)
    sp16 = sv.accept_params(tl16, dl16, vs.x, vs.ua, vs.us, cfg.temperature, vs.g, vs.cq, vs.cd, gmax, n16, tok16,
                            device_status=status)
    state.copy_(state0)
    t_a16 = median_us(lambda: check(lib.spec_accept_sample(C.byref(sp16), vs.ws_s.data_ptr(), vs.ws_s.numel(), sptr),
                                    "accept bf16"))
    a16_bytes = synth.algorithmic_bytes(cfg, seq_len, gamma)[1] // 2
    del tl16, dl16

    # ---- cache append (not part of the step above): the block's keys and values written behind the contexts
    n_kv = n_q * cfg.hkv * cfg.head_dim
    k_new = vs.up_bf16(synth.normal_bf16_bits(cfg.seed, 90, n_kv).reshape(n_q, cfg.hkv, cfg.head_dim))
    v_new = vs.up_bf16(synth.normal_bf16_bits(cfg.seed, 91, n_kv).reshape(n_q, cfg.hkv, cfg.head_dim))
    kp = sv.kv_append_params(k_new, v_new, vs.pool, vs.bt, vs.sl, vs.g, vs.cq, gmax, device_status=status)
    state.copy_(state0)
    t_ka = median_us(lambda: check(lib.spec_kv_append(C.byref(kp), sptr), "kv_append"))
    ka_bytes = int((gamma + 1).sum()) * cfg.hkv * cfg.head_dim * 2 * 2 * 2      # K and V, read and written

    # ---- --layers N: N caches of the same shape behind one block table; every step appends to all of them in
    # one launch and attends over each in turn (spec_verify_attn_layers), then accepts and updates once
    layers = None
    if args.layers > 1:
        pools, keep = [vs.pool], []
        for _ in range(args.layers - 1):
            kk, vv = vs.k_pool.clone(), vs.v_pool.clone()
            keep.append((kk, vv))
            pools.append(sv.spec_kv_pool_register(kk, vv))
        lp = sv.attn_layers_params([vs.q] * args.layers, [vs.o] * args.layers, pools, vs.bt, vs.sl, vs.g, vs.cq, gmax,
                                   vs.max_len, k_new=[k_new] * args.layers, v_new=[v_new] * args.layers,
                                   device_status=status)

        def layer_step(ev=None):
            state.copy_(state0, non_blocking=True)
            if ev is not None: ev[0].record(stream)
            check(lib.spec_verify_attn_layers(C.byref(lp), vs.ws_a.data_ptr(), vs.ws_a.numel(), sptr), "attn_layers")
            if ev is not None: ev[1].record(stream)
            check(lib.spec_accept_sample(C.byref(vs.sp), vs.ws_s.data_ptr(), vs.ws_s.numel(), sptr), "accept")
            check(lib.gamma_tune_update(C.byref(vs.gp), sptr), "gamma")
            if ev is not None: ev[2].record(stream)

        n_ls = max(3, min(args.steps, 20))
        for _ in range(3):
            layer_step()
        barrier()
        l_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_ls)]
        for it in range(n_ls):
            layer_step(l_ev[it])
        barrier()
        assert status.item() == 0, f"device status {status.item()}"
        t_layers = float(np.mean([e[0].elapsed_time(e[1]) for e in l_ev]))
        t_lstep = float(np.mean([e[0].elapsed_time(e[2]) for e in l_ev]))
        layers = {"n": args.layers, "steps": n_ls, "us_per_layer": 1e3 * t_layers / args.layers,
                  "step_us": 1e3 * t_lstep, "single_layer_attention_us": 1e3 * t_attn, "append_us": t_ka,
                  "gbs": args.layers * synth.algorithmic_bytes(cfg, seq_len, gamma)[0] / (t_layers * 1e-3) / 1e9}
        del keep, pools, lp
        torch.cuda.empty_cache()

    # ---- reduce over ranks: max time, sum of tokens
    (ms_total, e2e_ms), tokens_all = shard.reduce_timing([ms_total, e2e_ms], tokens, device=DEV)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_step = ms_total / args.steps
    attn_bytes, acc_bytes = synth.algorithmic_bytes(cfg, seq_len, gamma)
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    achieved = attn_bytes / (t_attn * 1e-3) / 1e9
    ratio = profiled_traffic_ratio() if cfg.name == "c5" else None
    wl_cfg = workload_config(cfg, gamma, "inputs larger than L2 (KV %.2f GB + logits %.2f GB per GPU), no flush"
                             % (attn_bytes / 1e9, acc_bytes / 1e9))
    wl_cfg["global_batch"] = global_batch
    line = {
        "metric": METRIC, "value": tokens_all / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": args.scaling if world > 1 else "weak", "vs_baseline": None,
        "dtype": "bf16 attention (fp32 accumulate), f32 logits, f64 decisions",
        "data": "synthetic", "config": wl_cfg,
        "step_us": {"attention": 1e3 * t_attn, "accept": 1e3 * t_acc, "gamma_update": 1e3 * t_gam},
        "us_per_batch_gamma": 1e3 * ms_step / float(gamma.sum()),
        "step_hbm": {"bytes": attn_bytes + acc_bytes, "gbs": (attn_bytes + acc_bytes) / (ms_step * 1e-3) / 1e9,
                     "frac_of_8tbs": (attn_bytes + acc_bytes) / (ms_step * 1e-3) / 8e12,
                     "frac_of_measured": (attn_bytes + acc_bytes) / (ms_step * 1e-3) / 1e9 / peak},
        "roofline": {"bound": "hbm", "kernel": "spec_verify_attn", "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None if ratio is None else ratio * attn_bytes},
        "accept_roofline": {"bound": "hbm", "achieved": acc_bytes / (t_acc * 1e-3) / 1e9, "peak": peak,
                            "unit": "GB/s", "frac": acc_bytes / (t_acc * 1e-3) / 1e9 / peak},
        "e2e": {"value": tokens_all / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches), "clocks": clocks,
        "draft_stop": {"what": "GammaTune+ early stop over the same draft rows, outside the timed step",
                       "us": t_ds, "bytes": ds_bytes, "gbs": ds_bytes / (t_ds * 1e-6) / 1e9,
                       "frac_of_measured": ds_bytes / (t_ds * 1e-6) / 1e9 / peak},
    }
    if clocks is not None and clocks.get("sm_mhz"):
        # the GPUs of a pool differ in the clock they hold; time x clock compares kernels across them
        line["step_us_x_sm_ghz"] = 1e3 * ms_step * clocks["sm_mhz"] / 1e3
    line["draft_step"] = {"what": "one drafting step with the confidence stop (a draft row per sequence: token, top "
                                  "probability, state), outside the timed step; includes two small fills",
                          "us": t_st, "bytes": st_bytes, "gbs": st_bytes / (t_st * 1e-6) / 1e9}
    line["accept_bf16_logits"] = {"what": "spec_accept_sample on the same logits stored as bf16, outside the timed step",
                                  "us": t_a16, "bytes": a16_bytes, "gbs": a16_bytes / (t_a16 * 1e-6) / 1e9,
                                  "frac_of_measured": a16_bytes / (t_a16 * 1e-6) / 1e9 / peak}
    line["kv_append"] = {"what": "the block's keys and values written into the paged cache, outside the timed step",
                         "us": t_ka, "bytes": ka_bytes}
    if layers is not None:
        layers["frac_of_measured"] = layers["gbs"] / peak
        line["layers"] = layers
    if world == 1 and not args.no_configs and args.workload == "c5" and args.batch is None:
        del vs
        torch.cuda.empty_cache()
        line["configs"] = config_lines(sv, torch, DEV, 50, peak)
        cfg, seq_len, gamma, cu_q, cu_d = workload_inputs(base_cfg, rank, args.batch, args.gamma, args.gamma_max)
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        n_seq = min(args.oracle_seqs or 64, B)
        sub, kv_s, q_s, li_s = sample_inputs(cfg, seq_len, gamma, cu_q, cu_d, n_seq)
        dt, otoks = oracle_step(sub, seq_len, gamma, cu_q, cu_d, kv_s, q_s, li_s, n_seq)
        line["cpu_baseline"] = {"value": otoks / dt, "unit": UNIT, "cores": oracle.num_threads(),
                                "kind": "oracle", "seconds": dt,
                                "sample": f"first {n_seq} of {B} sequences, whole step, once"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(args):
    """`--gpus N` without a launcher around this process: start N ranks of this same command (one per GPU, NCCL
    for the GPU arm) through torch.distributed.run on this node and pass their output through."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5", choices=sorted(synth.CONFIGS))
    ap.add_argument("--oracle-seqs", type=int, default=None,
                    help="sequences in the oracle's bounded sample (default 16 for cpu_baseline, 4 per step for --impl reference)")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gamma", type=int, default=None,
                    help="draft length of every sequence (default: the workload's own range)")
    ap.add_argument("--gamma-max", type=int, default=None, help="override the controller's upper bound")
    ap.add_argument("--evolve", type=int, default=0,
                    help="let the controller run this many steps before the timed ones (a GammaTune-driven gamma mix)")
    ap.add_argument("--layers", type=int, default=8,
                    help="also time steps that append to and attend over this many caches in turn (memory: one KV pool "
                         "each; 1 = off)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: every rank its own batch (weak), or one batch cut by cached tokens over the ranks (strong)")
    ap.add_argument("--no-configs", action="store_true", help="skip the step times of the workloads c1..c4")
    ap.add_argument("--batch", type=int, default=None,
                    help="override the workload's batch (smaller cases for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
