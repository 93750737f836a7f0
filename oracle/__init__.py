"""Float64 CPU oracle for the verify step -- TEST INFRASTRUCTURE ONLY.

This package wraps ``specverify_oracle.c`` (plain C, float64) with numpy
marshalling.  It defines what the CUDA library has to compute; it shares no
code with that library and neither imports the other.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.

The C file is compiled on first use with gcc (``-ffp-contract=off`` keeps the
controller's arithmetic as separately rounded IEEE binary64 operations).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "specverify_oracle.c")
_LIB = os.path.join(_HERE, "libspecverify_oracle.so")

MODE_FIXED = 0
MODE_GT_PROPOSED = 1
MODE_GT_LITERAL = 2

ACCEPT_TOL = 1e-6   # |u - ratio| below this: the accept decision is reported as a near tie
SAMPLE_TOL = 1e-9   # |u*W - CDF edge| below this fraction of W: the sampled token is a near tie


def build(force: bool = False) -> str:
    """Compile the oracle's C source into a shared object next to it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_cost_model.restype = ctypes.c_double
        _lib.oracle_cost_model.argtypes = [ctypes.c_double] * 4
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    """Threads the OpenMP loops use (OMP_NUM_THREADS, else all cores)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


# --------------------------------------------------------------------------- attention
def attn_row(q_row_bits, k_pool_bits, v_pool_bits, kv_strides, block_table_row, page_size,
             kv_head, n_keys, scale):
    """Softmax attention of one query row over keys 0..n_keys-1 (definition).

    q_row_bits: uint16 [D] bf16 bit patterns; pools: uint16 arrays; kv_strides:
    element strides (page, kv head, slot, dim).  Returns (o float64 [D], lse).
    """
    lib = _load()
    q = _c(q_row_bits, np.uint16)
    D = q.shape[0]
    st = _c(kv_strides, np.int64)
    bt = _c(block_table_row, np.int32)
    o = np.zeros(D, np.float64)
    lse = np.zeros(1, np.float64)
    lib.oracle_attn_row(_p(q), _p(k_pool_bits), _p(v_pool_bits), _p(st), _p(bt),
                        ctypes.c_int(page_size), ctypes.c_int(kv_head), ctypes.c_int(D),
                        ctypes.c_int(n_keys), ctypes.c_double(scale), _p(o), _p(lse))
    return o, float(lse[0])


def verify_attn(q_bits, k_pool_bits, v_pool_bits, kv_strides, block_table, seq_len, gamma, cu_q,
                hq, hkv, page_size, scale):
    """Attention of every draft-block row of a ragged batch.

    q_bits uint16 [sum R, hq, D].  Returns (o float64 [sum R, hq, D], lse [sum R, hq]).
    """
    lib = _load()
    q = _c(q_bits, np.uint16)
    n_rows, hq_, D = q.shape
    assert hq_ == hq
    assert k_pool_bits.dtype == np.uint16 and v_pool_bits.dtype == np.uint16
    st = _c(kv_strides, np.int64)
    bt = _c(block_table, np.int32)
    sl, g, cq = _c(seq_len, np.int32), _c(gamma, np.int32), _c(cu_q, np.int32)
    o = np.zeros((n_rows, hq, D), np.float64)
    lse = np.zeros((n_rows, hq), np.float64)
    lib.oracle_verify_attn(_p(q), _p(k_pool_bits), _p(v_pool_bits), _p(st), _p(bt),
                           ctypes.c_int64(bt.shape[1]), _p(sl), _p(g), _p(cq),
                           ctypes.c_int(len(sl)), ctypes.c_int(hq), ctypes.c_int(hkv),
                           ctypes.c_int(D), ctypes.c_int(page_size), ctypes.c_double(scale),
                           _p(o), _p(lse))
    return o, lse


def kv_append(k_new_bits, v_new_bits, k_pool_bits, v_pool_bits, kv_strides, block_table, seq_len, gamma,
              cu_q, page_size):
    """Write the draft block's keys and values behind each sequence's context.

    k_new_bits, v_new_bits uint16 [sum R, hkv, D]; the pools are flat or shaped uint16 arrays
    addressed through kv_strides (elements: page, head, slot, dim).  Returns modified copies of
    the two pools; the arguments are left alone.
    """
    lib = _load()
    kn, vn = _c(k_new_bits, np.uint16), _c(v_new_bits, np.uint16)
    n_rows, hkv, D = kn.shape
    assert vn.shape == kn.shape
    assert k_pool_bits.dtype == np.uint16 and v_pool_bits.dtype == np.uint16
    kp, vp = np.array(k_pool_bits, order="C", copy=True), np.array(v_pool_bits, order="C", copy=True)
    st = _c(kv_strides, np.int64)
    bt = _c(block_table, np.int32)
    sl, g, cq = _c(seq_len, np.int32), _c(gamma, np.int32), _c(cu_q, np.int32)
    lib.oracle_kv_append(_p(kn), _p(vn), _p(kp), _p(vp), _p(st), _p(bt), ctypes.c_int64(bt.shape[1]),
                         _p(sl), _p(g), _p(cq), ctypes.c_int(len(sl)), ctypes.c_int(hkv), ctypes.c_int(D),
                         ctypes.c_int(page_size))
    return kp, vp


# --------------------------------------------------------------------------- accept / resample
@dataclass
class AcceptResult:
    n_accepted: np.ndarray      # int32 [B]
    out_tokens: np.ndarray      # int32 [B, gamma_max+1]
    ratio: np.ndarray           # float64 [sum gamma] (NaN past the first rejection)
    logZ_p: np.ndarray          # float64 [sum R]
    logZ_q: np.ndarray          # float64 [sum gamma]
    accept_flag: np.ndarray     # uint8 [sum gamma]: |u - ratio| < ACCEPT_TOL
    alt_token: np.ndarray       # int32 [B]: the other legal token when sample_flag is set
    sample_flag: np.ndarray     # uint8 [B]
    resid_mass: np.ndarray      # float64 [B]: sum max(0, p-q) at a rejection, else NaN


def accept_sample(target_logits, draft_logits, draft_tokens, u_accept, u_sample, temperature,
                  gamma, cu_q, cu_d, gamma_max, force=None,
                  accept_tol=ACCEPT_TOL, sample_tol=SAMPLE_TOL) -> AcceptResult:
    """One accept / resample step for a ragged batch (see the C source for the rule)."""
    lib = _load()
    tl = _c(target_logits, np.float32)
    dl = _c(draft_logits, np.float32)
    V = tl.shape[1]
    assert dl.ndim == 2 and (dl.shape[0] == 0 or dl.shape[1] == V)
    g, cq, cd = _c(gamma, np.int32), _c(cu_q, np.int32), _c(cu_d, np.int32)
    B = len(g)
    x = _c(draft_tokens, np.int32)
    ua, us = _c(u_accept, np.float32), _c(u_sample, np.float32)
    T = np.broadcast_to(np.asarray(temperature, np.float32), (B,)).copy()
    n_d, n_q = int(cd[B]), int(cq[B])
    res = AcceptResult(
        n_accepted=np.zeros(B, np.int32), out_tokens=np.zeros((B, gamma_max + 1), np.int32),
        ratio=np.full(max(n_d, 1), np.nan), logZ_p=np.full(max(n_q, 1), np.nan),
        logZ_q=np.full(max(n_d, 1), np.nan), accept_flag=np.zeros(max(n_d, 1), np.uint8),
        alt_token=np.zeros(B, np.int32), sample_flag=np.zeros(B, np.uint8),
        resid_mass=np.zeros(B, np.float64))
    fptr = None
    if force is not None:
        force = _c(force, np.int8)
        fptr = _p(force)
    lib.oracle_accept_sample(_p(tl), _p(dl), ctypes.c_int64(V), ctypes.c_int(V), _p(x), _p(ua),
                             _p(us), _p(T), _p(g), _p(cq), _p(cd), ctypes.c_int(B),
                             ctypes.c_int(gamma_max), fptr, ctypes.c_double(accept_tol),
                             ctypes.c_double(sample_tol), _p(res.n_accepted), _p(res.out_tokens),
                             _p(res.ratio), _p(res.logZ_p), _p(res.logZ_q), _p(res.accept_flag),
                             _p(res.alt_token), _p(res.sample_flag), _p(res.resid_mass))
    res.ratio, res.logZ_q, res.accept_flag = res.ratio[:n_d], res.logZ_q[:n_d], res.accept_flag[:n_d]
    res.logZ_p = res.logZ_p[:n_q]
    return res


# --------------------------------------------------------------------------- GammaTune
def gamma_tune_init(batch: int, gamma0: int, gamma_max: int = 0, padded_rows: bool = False):
    """State for `batch` sequences: gamma_bar = gamma = gamma0, plus cu_q / cu_d."""
    lib = _load()
    gbar = np.zeros(batch, np.float64)
    g = np.zeros(batch, np.int32)
    cq = np.zeros(batch + 1, np.int32)
    cd = np.zeros(batch + 1, np.int32)
    lib.oracle_gamma_tune_init(_p(gbar), _p(g), _p(cq), _p(cd), ctypes.c_int(batch),
                               ctypes.c_int(gamma0), ctypes.c_int(gamma_max),
                               ctypes.c_int(int(padded_rows)))
    return gbar, g, cq, cd


def gamma_tune_update(n_accepted, gamma_bar, gamma, seq_len, eta, delta, gamma_min, gamma_max,
                      mode=MODE_GT_PROPOSED, padded_rows=False, n_drafted=None):
    """One controller update (Algorithm 1).  Returns NEW arrays
    (gamma_bar, gamma, seq_len, cu_q, cu_d); the inputs are not modified.
    n_drafted (GammaTune+): drafts actually produced this step, <= gamma."""
    lib = _load()
    A = _c(n_accepted, np.int32)
    B = len(A)
    gbar = np.array(gamma_bar, np.float64, copy=True)
    g = np.array(gamma, np.int32, copy=True)
    sl = np.array(seq_len, np.int32, copy=True)
    cq = np.zeros(B + 1, np.int32)
    cd = np.zeros(B + 1, np.int32)
    lib.oracle_gamma_tune_update(_p(A), _p(gbar), _p(g), _p(sl), _p(cq), _p(cd), ctypes.c_int(B),
                                 ctypes.c_double(eta), ctypes.c_double(delta),
                                 ctypes.c_int(gamma_min), ctypes.c_int(gamma_max),
                                 ctypes.c_int(mode), ctypes.c_int(int(padded_rows)),
                                 _p(_c(n_drafted, np.int32)) if n_drafted is not None else None)
    return gbar, g, sl, cq, cd


DRAFT_STOP_TOL = 1e-6


def draft_stop(draft_logits, temperature, tau, gamma, cu_d, tol=DRAFT_STOP_TOL):
    """GammaTune+ early stop (Section 4.2): returns (n_drafted [B], top_prob [n_d_rows], flag [n_d_rows])."""
    lib = _load()
    dl = _c(draft_logits, np.float32)
    g, cd = _c(gamma, np.int32), _c(cu_d, np.int32)
    B = len(g)
    T = np.broadcast_to(np.asarray(temperature, np.float32), (B,)).copy()
    n_d = int(cd[B])
    n = np.zeros(B, np.int32)
    top = np.full(max(n_d, 1), np.nan)
    flag = np.zeros(max(n_d, 1), np.uint8)
    lib.oracle_draft_stop(_p(dl), ctypes.c_int64(dl.shape[1] if dl.ndim == 2 else 0), ctypes.c_int(dl.shape[1]),
                          _p(T), ctypes.c_double(tau), _p(g), _p(cd), ctypes.c_int(B), ctypes.c_double(tol),
                          _p(n), _p(top), _p(flag))
    return n, top[:n_d], flag[:n_d]


def draft_step(draft_logits, temperature, tau, u, gamma, cu_d, n_drafted, active, draft_tokens, top_prob,
               tol=SAMPLE_TOL, conf_tol=DRAFT_STOP_TOL):
    """One drafting step with the confidence stop (Section 4.2).  n_drafted, active (int32 [B]), draft_tokens
    (int32 [n_d_rows]) and top_prob (float64 [n_d_rows]) are updated in place; returns (alt_token, sample_flag,
    conf_flag), each [B]."""
    lib = _load()
    dl = _c(draft_logits, np.float32)
    g, cd = _c(gamma, np.int32), _c(cu_d, np.int32)
    B = len(g)
    T = np.broadcast_to(np.asarray(temperature, np.float32), (B,)).copy()
    uu = _c(u, np.float32)
    for a, dt in ((n_drafted, np.int32), (active, np.int32), (draft_tokens, np.int32), (top_prob, np.float64)):
        assert a.dtype == dt and a.flags.c_contiguous
    alt = np.full(B, -1, np.int32)
    sflag = np.zeros(B, np.uint8)
    cflag = np.zeros(B, np.uint8)
    lib.oracle_draft_step(_p(dl), ctypes.c_int64(dl.shape[1]), ctypes.c_int(dl.shape[1]), _p(T), ctypes.c_double(tau),
                          _p(uu), _p(g), _p(cd), ctypes.c_int(B), ctypes.c_double(tol), ctypes.c_double(conf_tol),
                          _p(n_drafted), _p(active), _p(draft_tokens), _p(top_prob), _p(alt), _p(sflag), _p(cflag))
    return alt, sflag, cflag


def cost_model(n_tokens, alpha, gamma, c):
    """Inference cost of Eq. 2-6 in units of T_draft."""
    return float(_load().oracle_cost_model(n_tokens, alpha, gamma, c))
