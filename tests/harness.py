"""Shared helpers of the GPU parity tests: upload seeded inputs, call the CUDA
library through its binding, run the oracle on the same arrays, compare."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import oracle
from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth

DEV = "cuda:0"


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(DEV)


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(DEV).view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def workspace(nbytes: int) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=DEV)


# --------------------------------------------------------------------------- attention
@dataclass
class AttnCase:
    cfg: synth.VerifyConfig
    seq_len: np.ndarray
    gamma: np.ndarray
    cu_q: np.ndarray
    kv: synth.KVState
    q: np.ndarray          # uint16 [n_rows, hq, D]


def make_attn_case(cfg, seq_len=None, gamma=None, padded=False) -> AttnCase:
    sl, g = synth.draw_lengths(cfg)
    if seq_len is not None:
        sl = np.asarray(seq_len, np.int32)
    if gamma is not None:
        g = np.asarray(gamma, np.int32)
    cu_q, _ = synth.padded_offsets(cfg.batch, cfg.gamma_max) if padded else synth.prefix(g)
    kv = synth.make_kv(cfg, sl)
    q = synth.make_q(cfg, int(cu_q[-1]))
    return AttnCase(cfg, sl, g, cu_q, kv, q)


def run_attn_gpu(case: AttnCase, want_lse=True):
    cfg = case.cfg
    k, v = dev_bf16(case.kv.k_pool), dev_bf16(case.kv.v_pool)
    pool = sv.spec_kv_pool_register(k, v)
    q = dev_bf16(case.q)
    o = torch.zeros_like(q)
    lse = torch.zeros(q.shape[:2], dtype=torch.float32, device=DEV) if want_lse else None
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    max_len = int(case.seq_len.max())
    ws = workspace(sv.spec_verify_attn_workspace_bytes(cfg.batch, cfg.gamma_max, cfg.hq, cfg.hkv,
                                                       cfg.head_dim, max_len))
    bt = dev(case.kv.block_table)
    sv.spec_verify_attn(q, o, pool, bt, dev(case.seq_len), dev(case.gamma), dev(case.cu_q),
                        cfg.gamma_max, max_len, ws, lse=lse, device_status=status)
    torch.cuda.synchronize()
    o_f = synth.bf16_to_f32(bits_of(o)).astype(np.float64)
    return o_f, (lse.cpu().numpy().astype(np.float64) if want_lse else None), int(status.item())


def run_attn_oracle(case: AttnCase):
    cfg = case.cfg
    return oracle.verify_attn(case.q, case.kv.k_pool, case.kv.v_pool, case.kv.strides,
                              case.kv.block_table, case.seq_len, case.gamma, case.cu_q, cfg.hq,
                              cfg.hkv, cfg.page_size, float(np.float32(cfg.head_dim ** -0.5)))


def used_rows(gamma, cu_q):
    return np.concatenate([np.arange(cu_q[b], cu_q[b] + gamma[b] + 1) for b in range(len(gamma))])


ATTN_ATOL = 2e-2        # bf16 attention outputs, absolute


def attn_allowed(o_ref):
    """2e-2 absolute.  A bf16 value of magnitude >= 4 is a multiple of 2^-5, so its correctly
    rounded result can already sit 0.0156 from the exact one; for those elements (reached only
    by the peaky stress cases) half a bf16 ulp of the reference is added to the bound."""
    a = np.abs(o_ref)
    return ATTN_ATOL + np.where(a >= 4.0, a * 2.0 ** -8, 0.0)


SUM_RTOL = 1e-5         # fp32 softmax sums, relative


def check_attn(case: AttnCase):
    o_gpu, lse_gpu, status = run_attn_gpu(case)
    o_ref, lse_ref = run_attn_oracle(case)
    rows = used_rows(case.gamma, case.cu_q)
    assert status == 0, f"device status {status}"
    diff = np.abs(o_gpu[rows] - o_ref[rows])
    err = diff.max()
    w = np.unravel_index(np.argmax(diff - attn_allowed(o_ref[rows])), diff.shape)
    assert (diff <= attn_allowed(o_ref[rows])).all(), \
        f"attention output error {diff[w]} at used-row {w}: gpu {o_gpu[rows][w]} vs oracle {o_ref[rows][w]}"
    # softmax sums: exp(lse) relative error
    rel = np.abs(np.expm1(lse_gpu[rows] - lse_ref[rows])).max()
    assert rel <= SUM_RTOL, f"softmax sum relative error {rel}"
    return err, rel


# --------------------------------------------------------------------------- accept / resample
@dataclass
class AcceptOut:
    n_accepted: np.ndarray
    out_tokens: np.ndarray
    ratio: np.ndarray
    logZ_p: np.ndarray
    logZ_q: np.ndarray
    flag_count: int
    status: int


def bf16_rounded(li: synth.LogitInputs) -> synth.LogitInputs:
    """The same inputs with every logit rounded to bf16 (held as float32: the oracle's view of bf16 logits)."""
    r = lambda x: synth.bf16_to_f32(synth.bf16_bits(x)).reshape(x.shape)
    return synth.LogitInputs(r(li.target_logits), r(li.draft_logits), li.draft_tokens, li.u_accept, li.u_sample)


def run_accept_gpu(li: synth.LogitInputs, temperature, gamma, cu_q, cu_d, gamma_max,
                   temperature_per_seq=None, bf16=False) -> AcceptOut:
    """bf16: the logits (already bf16-representable, see bf16_rounded) go to the device as bf16 tensors."""
    B = len(gamma)
    V = li.target_logits.shape[1]
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    ldt = torch.bfloat16 if bf16 else torch.float32
    tl = dev(li.target_logits).to(ldt)
    dl = dev(li.draft_logits).to(ldt) if n_d > 0 else torch.zeros((1, V), dtype=ldt, device=DEV)
    x = dev(li.draft_tokens) if n_d > 0 else torch.zeros(1, dtype=torch.int32, device=DEV)
    ua = dev(li.u_accept) if n_d > 0 else torch.zeros(1, dtype=torch.float32, device=DEV)
    us = dev(li.u_sample)
    n_acc = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    out = torch.full((B, gamma_max + 1), -7, dtype=torch.int32, device=DEV)
    ratio = torch.full((max(n_d, 1),), float("nan"), dtype=torch.float64, device=DEV)
    lzp = torch.full((n_q,), float("nan"), dtype=torch.float64, device=DEV)
    lzq = torch.full((max(n_d, 1),), float("nan"), dtype=torch.float64, device=DEV)
    flags = torch.zeros(1, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ws = workspace(sv.spec_accept_sample_workspace_bytes(B, gamma_max, V))
    tps = dev(np.asarray(temperature_per_seq, np.float32)) if temperature_per_seq is not None else None
    sv.spec_accept_sample(tl, dl, x, ua, us, float(temperature), dev(gamma), dev(cu_q), dev(cu_d),
                          gamma_max, n_acc, out, ws, ratio=ratio, logZ_p=lzp, logZ_q=lzq,
                          flag_count=flags, device_status=status, temperature_per_seq=tps)
    torch.cuda.synchronize()
    return AcceptOut(n_acc.cpu().numpy(), out.cpu().numpy(), ratio.cpu().numpy()[:n_d],
                     lzp.cpu().numpy(), lzq.cpu().numpy()[:n_d], int(flags.item()),
                     int(status.item()))


def compare_accept(gpu: AcceptOut, li: synth.LogitInputs, temperature, gamma, cu_q, cu_d, gamma_max):
    """Bit-exact comparison of accepted counts and emitted tokens with the oracle.

    A position the ORACLE reports as a near tie (|u - ratio| < 1e-6) may go
    either way: the oracle is re-run with the device's decision forced there
    and the comparison continues.  A sampled token the oracle reports as a
    near tie may be either of the two neighbouring tokens.  Returns the
    numbers of positions / samples that needed this."""
    B = len(gamma)
    T = np.broadcast_to(np.asarray(temperature, np.float32), (B,))
    ref = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept,
                               li.u_sample, T, gamma, cu_q, cu_d, gamma_max)
    n_flag_pos = n_flag_tok = 0
    force = None
    for _ in range(4):
        bad = np.flatnonzero(gpu.n_accepted != ref.n_accepted)
        if len(bad) == 0:
            break
        force = np.full(max(int(cu_d[-1]), 1), -1, np.int8) if force is None else force
        for b in bad:
            i = int(min(gpu.n_accepted[b], ref.n_accepted[b]))
            assert i < gamma[b] and ref.accept_flag[cu_d[b] + i], \
                f"sequence {b}: accepted {gpu.n_accepted[b]} vs oracle {ref.n_accepted[b]}, position {i} is not a near tie"
            force[cu_d[b] + i] = 1 if gpu.n_accepted[b] > i else 0
            n_flag_pos += 1
        ref = oracle.accept_sample(li.target_logits, li.draft_logits, li.draft_tokens, li.u_accept,
                                   li.u_sample, T, gamma, cu_q, cu_d, gamma_max, force=force)
    np.testing.assert_array_equal(gpu.n_accepted, ref.n_accepted)
    for b in range(B):
        if np.array_equal(gpu.out_tokens[b], ref.out_tokens[b]):
            continue
        n = ref.n_accepted[b]
        alt = ref.out_tokens[b].copy()
        alt[n] = ref.alt_token[b]
        assert ref.sample_flag[b] and np.array_equal(gpu.out_tokens[b], alt), \
            f"sequence {b}: tokens {gpu.out_tokens[b]} vs oracle {ref.out_tokens[b]} (alt {ref.alt_token[b]})"
        n_flag_tok += 1
    return ref, n_flag_pos, n_flag_tok


def check_accept(li, temperature, gamma, cu_q, cu_d, gamma_max, temperature_per_seq=None, bf16=False):
    T = temperature_per_seq if temperature_per_seq is not None else temperature
    gpu = run_accept_gpu(li, temperature, gamma, cu_q, cu_d, gamma_max, temperature_per_seq, bf16)
    assert gpu.status == 0, f"device status {gpu.status}"
    ref, n_pos, n_tok = compare_accept(gpu, li, T, gamma, cu_q, cu_d, gamma_max)
    # softmax sums (fp32 exponentials): Z relative error <= 1e-5, i.e. |d lnZ| <= 1e-5
    ok_p = np.isfinite(ref.logZ_p)
    if ok_p.any():
        assert np.abs(np.expm1(gpu.logZ_p[ok_p] - ref.logZ_p[ok_p])).max() <= SUM_RTOL
    ok_q = np.isfinite(ref.logZ_q)
    if ok_q.any():
        assert np.abs(np.expm1(gpu.logZ_q[ok_q] - ref.logZ_q[ok_q])).max() <= SUM_RTOL
    ok_r = np.isfinite(ref.ratio) & np.isfinite(gpu.ratio)
    if ok_r.any():
        assert np.abs(gpu.ratio[ok_r] - ref.ratio[ok_r]).max() <= 1e-6
    return gpu, ref, n_pos, n_tok
