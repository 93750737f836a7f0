"""Benchmark of the verify step (attention + accept/resample + gamma update).

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload c5]

One step = one pass of the whole hot path over one batch of seeded synthetic
input.  The default workload is the largest configuration (Llama-3.1-70B-shaped:
batch 128, 64q/8kv heads, ragged contexts 512..16384, V = 128256, gamma = 16 for
every sequence, temperature 1, noise sigma 1).  The controller state is reset to
the same values before every step (one small device-to-device copy inside the
timed region), so that every timed step does the same work on the same inputs.

N > 1: one process per GPU (torchrun); each rank runs its own batch (sequences
are independent, no data-path collective); value = all ranks' tokens / max time.

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
# DRAM traffic of the attention main kernel per algorithmic byte, from one ncu capture
# (dram__bytes_read.sum + dram__bytes_write.sum of attn_tq_kernel<1> on the c5 shapes at batch
# 32: 1.0551 GB + 0.0180 GB for 1 056 358 400 algorithmic bytes).  The workload there was cut
# down to keep the capture short; traffic grows with the KV bytes, so the full launch's figure
# is this ratio times its algorithmic bytes.  Set to None whenever the kernel changes.
NCU_ATTN_TRAFFIC_RATIO = 1.0159


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
    cfg, seq_len, gamma, cu_q, cu_d = workload_inputs(base_cfg, rank, args.batch, args.gamma, args.gamma_max)
    B, gmax = cfg.batch, cfg.gamma_max
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    reserve = (2 + args.evolve) * (gmax + 1)
    kv = synth.make_kv(cfg, seq_len, reserve_tokens=reserve)
    q_np = synth.make_q(cfg, n_q)
    li = synth.make_logits(cfg, gamma, cu_q, cu_d)

    def up(a):
        return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)

    def up_bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)

    def pin(a):
        return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()

    k_pool, v_pool = up_bf16(kv.k_pool), up_bf16(kv.v_pool)
    pool = sv.spec_kv_pool_register(k_pool, v_pool)
    bt = up(kv.block_table)
    max_len = int(seq_len.max()) + reserve
    # host (pinned) copies of the per-step inputs for the end-to-end leg
    q_h = torch.from_numpy(q_np.view(np.int16)).view(torch.bfloat16).pin_memory()
    tl_h, dl_h = pin(li.target_logits), pin(li.draft_logits)
    x_h, ua_h, us_h = pin(li.draft_tokens), pin(li.u_accept), pin(li.u_sample)
    # device-resident inputs
    q = q_h.to(DEV)
    o = torch.zeros_like(q)
    tl, dl = tl_h.to(DEV), dl_h.to(DEV)
    x, ua, us = x_h.to(DEV), ua_h.to(DEV), us_h.to(DEV)
    n_acc = torch.zeros(B, dtype=torch.int32, device=DEV)
    toks = torch.zeros((B, gmax + 1), dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # controller state in one buffer so that one copy resets it: gbar | gamma | seq_len | cu_q | cu_d
    nb = 8 * B + 4 * B + 4 * B + 4 * (B + 1) + 4 * (B + 1)
    state = torch.zeros(nb, dtype=torch.uint8, device=DEV)
    off = 0
    gbar = state[off:off + 8 * B].view(torch.float64); off += 8 * B
    g = state[off:off + 4 * B].view(torch.int32); off += 4 * B
    sl = state[off:off + 4 * B].view(torch.int32); off += 4 * B
    cq = state[off:off + 4 * (B + 1)].view(torch.int32); off += 4 * (B + 1)
    cd = state[off:off + 4 * (B + 1)].view(torch.int32)
    gbar.copy_(up(gamma.astype(np.float64)))
    g.copy_(up(gamma)); sl.copy_(up(seq_len)); cq.copy_(up(cu_q)); cd.copy_(up(cu_d))
    state0 = state.clone()
    gcfg = sv.GammaConfig(GT["eta"], GT["delta"], GT["gamma_min"], gmax, sv.SV_GT_PROPOSED, True)
    ws_a = torch.empty(max(256, sv.spec_verify_attn_workspace_bytes(B, gmax, cfg.hq, cfg.hkv, cfg.head_dim,
                                                                    max_len)), dtype=torch.uint8, device=DEV)
    ws_s = torch.empty(max(256, sv.spec_accept_sample_workspace_bytes(B, gmax, cfg.vocab)), dtype=torch.uint8,
                       device=DEV)
    ap = sv.attn_params(q, o, pool, bt, sl, g, cq, gmax, max_len, device_status=status)
    sp = sv.accept_params(tl, dl, x, ua, us, cfg.temperature, g, cq, cd, gmax, n_acc, toks,
                          device_status=status)
    gp = sv.gamma_params(n_acc, gbar, g, sl, cq, cd, gcfg, device_status=status)
    lib = sv.load()
    import ctypes as C
    stream = torch.cuda.current_stream()
    sptr = C.c_void_p(stream.cuda_stream)

    def check(st, what):
        if st != 0:
            raise RuntimeError(f"{what}: {sv.status_str(st)}")

    def step(ev=None):
        state.copy_(state0, non_blocking=True)
        if ev is not None: ev[0].record(stream)
        check(lib.spec_verify_attn(C.byref(ap), ws_a.data_ptr(), ws_a.numel(), sptr), "attn")
        if ev is not None: ev[1].record(stream)
        check(lib.spec_accept_sample(C.byref(sp), ws_s.data_ptr(), ws_s.numel(), sptr), "accept")
        if ev is not None: ev[2].record(stream)
        check(lib.gamma_tune_update(C.byref(gp), sptr), "gamma")
        if ev is not None: ev[3].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.evolve > 0:
        # --evolve N: the controller runs N steps on its own acceptance counts first (no reset), and
        # the timed steps start from the state it reached: a GammaTune-driven mix of draft lengths
        # instead of gamma_max everywhere (the logit rows of a slab beyond a sequence's gamma are unused).
        state.copy_(state0)
        for _ in range(args.evolve):
            check(lib.spec_verify_attn(C.byref(ap), ws_a.data_ptr(), ws_a.numel(), sptr), "attn")
            check(lib.spec_accept_sample(C.byref(sp), ws_s.data_ptr(), ws_s.numel(), sptr), "accept")
            check(lib.gamma_tune_update(C.byref(gp), sptr), "gamma")
        torch.cuda.synchronize()
        state0 = state.clone()
        gamma = g.cpu().numpy().copy()
        seq_len = sl.cpu().numpy().copy()
    for _ in range(args.warmup):
        step()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    e_begin, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = sv.sv_launch_count()
    tokens = 0
    barrier()
    e_begin.record(stream)
    for it in range(args.steps):
        step(evs[it])
    e_end.record(stream)
    barrier()
    launches = sv.sv_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms_total = e_begin.elapsed_time(e_end)
    tokens = int((n_acc + 1).sum().item())          # identical every step (same inputs, same state)
    assert status.item() == 0, f"device status {status.item()}"
    t_attn = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    t_acc = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    t_gam = float(np.mean([e[2].elapsed_time(e[3]) for e in evs]))

    # ---- end to end through the host-buffer entry point
    n_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    tok_h = torch.zeros((B, gmax + 1), dtype=torch.int32).pin_memory()
    g_h = torch.zeros(B, dtype=torch.int32).pin_memory()
    o_h = torch.zeros(q_h.shape, dtype=torch.bfloat16).pin_memory()
    io = sv.step_host_io(q_h, tl_h, dl_h, x_h, ua_h, us_h, n_q, n_d, n_h, tok_h, g_h, o_h)
    h2d = sum(t.numel() * t.element_size() for t in (q_h, tl_h, dl_h, x_h, ua_h, us_h))
    d2h = sum(t.numel() * t.element_size() for t in (n_h, tok_h, g_h, o_h))
    e2e_steps = max(3, min(args.steps, args.e2e_steps))

    def e2e_step():
        state.copy_(state0, non_blocking=True)
        check(lib.spec_verify_step_host(C.byref(io), C.byref(ap), ws_a.data_ptr(), ws_a.numel(), C.byref(sp),
                                        ws_s.data_ptr(), ws_s.numel(), C.byref(gp), sptr), "step_host")
        stream.synchronize()                           # the caller reads the host results every step

    for _ in range(2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_tokens = int((n_h + 1).sum().item())
    assert e2e_tokens == tokens

    # ---- GammaTune+ early stop (not part of the step above): one streaming pass over the draft rows
    n_dr = torch.zeros(B, dtype=torch.int32, device=DEV)
    ws_d = torch.empty(max(256, sv.spec_draft_stop_workspace_bytes(B, gmax, cfg.vocab)), dtype=torch.uint8,
                       device=DEV)
    dp = sv.draft_stop_params(dl, cfg.temperature, 0.5, g, cd, gmax, n_dr, device_status=status)
    state.copy_(state0)
    ds_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]
    for _ in range(3):
        check(lib.spec_draft_stop(C.byref(dp), ws_d.data_ptr(), ws_d.numel(), sptr), "draft_stop")
    for e_a, e_b in ds_ev:
        e_a.record(stream)
        check(lib.spec_draft_stop(C.byref(dp), ws_d.data_ptr(), ws_d.numel(), sptr), "draft_stop")
        e_b.record(stream)
    barrier()
    t_ds = float(np.median([e_a.elapsed_time(e_b) for e_a, e_b in ds_ev]))
    ds_bytes = int(gamma.sum()) * cfg.vocab * 4

    # ---- cache append (not part of the step above): the block's keys and values written behind the contexts
    n_kv = n_q * cfg.hkv * cfg.head_dim
    k_new = up_bf16(synth.normal_bf16_bits(cfg.seed, 90, n_kv).reshape(n_q, cfg.hkv, cfg.head_dim))
    v_new = up_bf16(synth.normal_bf16_bits(cfg.seed, 91, n_kv).reshape(n_q, cfg.hkv, cfg.head_dim))
    kp = sv.kv_append_params(k_new, v_new, pool, bt, sl, g, cq, gmax, device_status=status)
    state.copy_(state0)
    ka_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(10)]
    for _ in range(3):
        check(lib.spec_kv_append(C.byref(kp), sptr), "kv_append")
    for e_a, e_b in ka_ev:
        e_a.record(stream)
        check(lib.spec_kv_append(C.byref(kp), sptr), "kv_append")
        e_b.record(stream)
    barrier()
    t_ka = float(np.median([e_a.elapsed_time(e_b) for e_a, e_b in ka_ev]))
    ka_bytes = int((gamma + 1).sum()) * cfg.hkv * cfg.head_dim * 2 * 2 * 2      # K and V, read and written

    # ---- --layers N: N caches of the same shape behind one block table; every step appends to and
    # attends over each of them in turn, then accepts and updates once (a model's worth of layers)
    layers = None
    if args.layers > 1:
        pools = [pool]
        keep = []
        for _ in range(args.layers - 1):
            kk, vv = k_pool.clone(), v_pool.clone()
            keep.append((kk, vv))
            pools.append(sv.spec_kv_pool_register(kk, vv))
        aps = [sv.attn_params(q, o, pl, bt, sl, g, cq, gmax, max_len, device_status=status) for pl in pools]
        kps = [sv.kv_append_params(k_new, v_new, pl, bt, sl, g, cq, gmax, device_status=status) for pl in pools]

        def layer_step(ev=None):
            state.copy_(state0, non_blocking=True)
            if ev is not None: ev[0].record(stream)
            for a_l, k_l in zip(aps, kps):
                check(lib.spec_kv_append(C.byref(k_l), sptr), "kv_append")
                check(lib.spec_verify_attn(C.byref(a_l), ws_a.data_ptr(), ws_a.numel(), sptr), "attn")
            if ev is not None: ev[1].record(stream)
            check(lib.spec_accept_sample(C.byref(sp), ws_s.data_ptr(), ws_s.numel(), sptr), "accept")
            check(lib.gamma_tune_update(C.byref(gp), sptr), "gamma")
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
                  "step_us": 1e3 * t_lstep,
                  "gbs": args.layers * synth.algorithmic_bytes(cfg, seq_len, gamma)[0] / (t_layers * 1e-3) / 1e9}

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
    line = {
        "metric": METRIC, "value": tokens_all / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 attention (fp32 accumulate), f32 logits, f64 decisions",
        "data": "synthetic",
        "config": workload_config(cfg, gamma, "inputs larger than L2 (KV %.2f GB + logits %.2f GB per GPU), no flush"
                                  % (attn_bytes / 1e9, acc_bytes / 1e9)),
        "step_us": {"attention": 1e3 * t_attn, "accept": 1e3 * t_acc, "gamma_update": 1e3 * t_gam},
        "us_per_batch_gamma": 1e3 * ms_step / float(gamma.sum()),
        "step_hbm": {"bytes": attn_bytes + acc_bytes, "gbs": (attn_bytes + acc_bytes) / (ms_step * 1e-3) / 1e9,
                     "frac_of_8tbs": (attn_bytes + acc_bytes) / (ms_step * 1e-3) / 8e12,
                     "frac_of_measured": (attn_bytes + acc_bytes) / (ms_step * 1e-3) / 1e9 / peak},
        "roofline": {"bound": "hbm", "kernel": "spec_verify_attn", "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (None if NCU_ATTN_TRAFFIC_RATIO is None or cfg.name != "c5"
                                 else NCU_ATTN_TRAFFIC_RATIO * attn_bytes)},
        "accept_roofline": {"bound": "hbm", "achieved": acc_bytes / (t_acc * 1e-3) / 1e9, "peak": peak,
                            "unit": "GB/s", "frac": acc_bytes / (t_acc * 1e-3) / 1e9 / peak},
        "e2e": {"value": tokens_all / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches), "clocks": clocks,
        "draft_stop": {"what": "GammaTune+ early stop over the same draft rows, outside the timed step",
                       "us": 1e3 * t_ds, "bytes": ds_bytes, "gbs": ds_bytes / (t_ds * 1e-3) / 1e9,
                       "frac_of_measured": ds_bytes / (t_ds * 1e-3) / 1e9 / peak},
    }
    line["kv_append"] = {"what": "the block's keys and values written into the paged cache, outside the timed step",
                         "us": 1e3 * t_ka, "bytes": ka_bytes}
    if layers is not None:
        layers["frac_of_measured"] = layers["gbs"] / peak
        line["layers"] = layers
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        n_seq = min(args.oracle_seqs or 16, B)
        dt, otoks = oracle_step(cfg, seq_len, gamma, cu_q, cu_d, kv, q_np, li, n_seq)
        line["cpu_baseline"] = {"value": otoks / dt, "unit": UNIT, "cores": oracle.num_threads(),
                                "kind": "oracle", "seconds": dt,
                                "sample": f"first {n_seq} of {B} sequences, whole step, once"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


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
    ap.add_argument("--layers", type=int, default=1,
                    help="also time steps that append to and attend over this many caches in turn (memory: one KV pool each)")
    ap.add_argument("--batch", type=int, default=None,
                    help="override the workload's batch (smaller cases for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
