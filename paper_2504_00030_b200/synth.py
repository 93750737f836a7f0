"""Seeded synthetic inputs for the verify step.

Numpy only.  This module produces inputs (KV pools, block tables, queries,
logits, draft tokens, uniforms) with the shapes and value distributions of the
paper's four target/draft pairs; it contains none of the verify step's own
arithmetic (no softmax, no acceptance rule, no controller), so the CUDA
library's callers and the CPU oracle's callers can both use it.

Random streams are Philox generators keyed by (seed, tensor id, chunk), so a
tensor does not depend on how many threads filled it or on what else was drawn.
"""
from __future__ import annotations

import concurrent.futures as _cf
import os
from dataclasses import dataclass, replace

import numpy as np

PAGE_SIZE = 16
_CHUNK = 1 << 22

# tensor ids for the Philox key
_T_K, _T_V, _T_Q, _T_BASE, _T_NOISE, _T_GUMBEL, _T_UACC, _T_USAMP, _T_PERM, _T_LEN, _T_GAMMA, _T_MIX = range(12)


def _rng(seed: int, tensor: int, chunk: int = 0, step: int = 0) -> np.random.Generator:
    key = ((int(seed) << 32) ^ (int(step) << 8) ^ int(tensor)) & 0xFFFFFFFFFFFFFFFF
    return np.random.Generator(np.random.Philox(key=[key, int(chunk)]))


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float32, exact."""
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _fill_chunks(n: int, fn, out: np.ndarray, threads: int | None = None):
    n_chunks = (n + _CHUNK - 1) // _CHUNK
    threads = threads or min(16, os.cpu_count() or 1)

    def work(c):
        lo, hi = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        out[lo:hi] = fn(c, hi - lo)

    if n_chunks <= 1 or threads <= 1:
        for c in range(n_chunks):
            work(c)
    else:
        with _cf.ThreadPoolExecutor(threads) as ex:
            list(ex.map(work, range(n_chunks)))
    return out


def normal_f32(seed: int, tensor: int, n: int, sigma: float = 1.0, step: int = 0) -> np.ndarray:
    """n float32 draws of N(0, sigma^2) (sigma is the standard deviation)."""
    out = np.empty(n, np.float32)

    def fn(c, m):
        x = _rng(seed, tensor, c, step).standard_normal(m, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        return x

    return _fill_chunks(n, fn, out)


def normal_bf16_bits(seed: int, tensor: int, n: int, sigma: float = 1.0, step: int = 0) -> np.ndarray:
    """n bf16 values (as uint16 bit patterns) rounded from N(0, sigma^2) float32 draws."""
    out = np.empty(n, np.uint16)

    def fn(c, m):
        x = _rng(seed, tensor, c, step).standard_normal(m, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        return bf16_bits(x)

    return _fill_chunks(n, fn, out)


def uniform_f32(seed: int, tensor: int, n: int, step: int = 0) -> np.ndarray:
    """n float32 uniforms in [0, 1)."""
    return _rng(seed, tensor, 0, step).random(n, dtype=np.float32)


# --------------------------------------------------------------------------- configurations
@dataclass(frozen=True)
class VerifyConfig:
    """One verify-step workload (shapes follow a target model of the paper)."""
    name: str
    batch: int
    hq: int
    hkv: int
    head_dim: int
    vocab: int
    ctx_lo: int                # KV length (draft block included), drawn uniformly in [ctx_lo, ctx_hi]
    ctx_hi: int
    gamma_lo: int              # per-sequence draft length, drawn uniformly in [gamma_lo, gamma_hi]
    gamma_hi: int
    gamma_max: int             # controller upper bound / row padding
    temperature: float
    sigma_noise: float         # std of (target - draft) logit noise
    sigma_draft: float = 2.0   # std of draft logits
    q_scale: float = 1.0       # std of the queries
    page_size: int = PAGE_SIZE
    seed: int = 20250400

    @property
    def group(self) -> int:
        return self.hq // self.hkv


CONFIGS = {
    # tiny, vicuna-68m-shaped
    "c1": VerifyConfig("c1", 1, 12, 12, 64, 32000, 128, 128, 4, 4, 4, 1.0, 0.5, seed=20250401),
    # vicuna-7B-shaped, gamma driven 1..8 by the controller
    "c2": VerifyConfig("c2", 1, 32, 32, 128, 32000, 2048, 2048, 1, 8, 8, 1.0, 1.0, seed=20250402),
    # Llama-3.1-8B-shaped
    "c3": VerifyConfig("c3", 16, 32, 8, 128, 128256, 1024, 8192, 2, 10, 10, 0.7, 0.8, seed=20250403),
    # vicuna-13B-shaped
    "c4": VerifyConfig("c4", 64, 40, 40, 128, 32000, 4096, 4096, 1, 12, 12, 1.0, 0.5, seed=20250404),
    # Llama-3.1-70B-shaped (the largest)
    "c5": VerifyConfig("c5", 128, 64, 8, 128, 128256, 512, 16384, 16, 16, 16, 1.0, 1.0, seed=20250405),
}


def scaled(cfg: VerifyConfig, **kw) -> VerifyConfig:
    """A copy of a configuration with some fields replaced (smaller test cases)."""
    return replace(cfg, **kw)


# --------------------------------------------------------------------------- batch structure
def draw_lengths(cfg: VerifyConfig, step: int = 0):
    """seq_len [B] (KV length including the draft block) and gamma [B], seeded."""
    r = _rng(cfg.seed, _T_LEN, 0, step)
    seq_len = r.integers(cfg.ctx_lo, cfg.ctx_hi + 1, size=cfg.batch).astype(np.int32)
    r = _rng(cfg.seed, _T_GAMMA, 0, step)
    gamma = r.integers(cfg.gamma_lo, cfg.gamma_hi + 1, size=cfg.batch).astype(np.int32)
    seq_len = np.maximum(seq_len, gamma + 1)
    return seq_len, gamma


def prefix(gamma: np.ndarray):
    """cu_q (prefix sums of gamma+1) and cu_d (prefix sums of gamma), int32 [B+1]."""
    cu_q = np.zeros(len(gamma) + 1, np.int32)
    cu_d = np.zeros(len(gamma) + 1, np.int32)
    cu_q[1:] = np.cumsum(gamma + 1)
    cu_d[1:] = np.cumsum(gamma)
    return cu_q, cu_d


def padded_offsets(batch: int, gamma_max: int):
    """Row offsets when every sequence owns a fixed slab of gamma_max+1 / gamma_max rows."""
    cu_q = (np.arange(batch + 1) * (gamma_max + 1)).astype(np.int32)
    cu_d = (np.arange(batch + 1) * gamma_max).astype(np.int32)
    return cu_q, cu_d


@dataclass
class KVState:
    k_pool: np.ndarray        # uint16 [n_pages, hkv, page_size, D] bf16 bits
    v_pool: np.ndarray
    block_table: np.ndarray   # int32 [B, max_pages]; unused entries are -1
    strides: np.ndarray       # int64 [4] element strides (page, head, slot, dim)


def make_kv(cfg: VerifyConfig, seq_len: np.ndarray, reserve_tokens: int = 0,
            extra_pages: int = 3) -> KVState:
    """Paged bf16 KV pool ~N(0,1) and a block table of scattered physical pages.

    Each sequence gets pages for seq_len + reserve_tokens tokens; the physical
    page ids are a seeded random permutation of the pool, so consecutive
    logical pages are not neighbours in memory.
    """
    ps = cfg.page_size
    pages_per_seq = (seq_len.astype(np.int64) + reserve_tokens + ps - 1) // ps
    n_pages = int(pages_per_seq.sum()) + extra_pages
    n_el = n_pages * cfg.hkv * ps * cfg.head_dim
    shape = (n_pages, cfg.hkv, ps, cfg.head_dim)
    k_pool = normal_bf16_bits(cfg.seed, _T_K, n_el).reshape(shape)
    v_pool = normal_bf16_bits(cfg.seed, _T_V, n_el).reshape(shape)
    perm = _rng(cfg.seed, _T_PERM).permutation(n_pages).astype(np.int32)
    max_pages = int(pages_per_seq.max())
    bt = np.full((cfg.batch, max_pages), -1, np.int32)
    at = 0
    for b in range(cfg.batch):
        n = int(pages_per_seq[b])
        bt[b, :n] = perm[at:at + n]
        at += n
    strides = np.array([cfg.hkv * ps * cfg.head_dim, ps * cfg.head_dim, cfg.head_dim, 1], np.int64)
    return KVState(k_pool, v_pool, bt, strides)


def make_q(cfg: VerifyConfig, n_rows: int, step: int = 0) -> np.ndarray:
    """Queries [n_rows, hq, D] as bf16 bits, N(0, q_scale^2)."""
    n = n_rows * cfg.hq * cfg.head_dim
    return normal_bf16_bits(cfg.seed, _T_Q, n, cfg.q_scale, step).reshape(n_rows, cfg.hq, cfg.head_dim)


@dataclass
class LogitInputs:
    target_logits: np.ndarray   # float32 [n_q_rows, V]
    draft_logits: np.ndarray    # float32 [n_d_rows, V]
    draft_tokens: np.ndarray    # int32 [n_d_rows]
    u_accept: np.ndarray        # float32 [n_d_rows]
    u_sample: np.ndarray        # float32 [B]


def mixture_rows(cfg: VerifyConfig, n_rows: int, step: int, hard_prob: float,
                 easy=(3.0, 0.3), hard=(1.0, 2.0)):
    """Per-row (sigma_draft, sigma_noise) for a workload whose positions differ in difficulty.

    Every row is "hard" with probability hard_prob (seeded) and "easy" otherwise.  An easy
    position has a peaked draft distribution (large logit spread) that the target nearly
    shares (small noise); a hard one a flat draft distribution far from the target's.  This
    models the premise of confidence-guided drafting (paper Section 4.2): where the draft
    model is unsure, its token is likely to be rejected.  Returns two float32 arrays [n_rows]."""
    is_hard = _rng(cfg.seed, _T_MIX, 0, step).random(n_rows) < hard_prob
    sd = np.where(is_hard, hard[0], easy[0]).astype(np.float32)
    sn = np.where(is_hard, hard[1], easy[1]).astype(np.float32)
    return sd, sn


def make_logits(cfg: VerifyConfig, gamma: np.ndarray, cu_q: np.ndarray, cu_d: np.ndarray,
                step: int = 0, sigma_noise: float | None = None,
                temperature: float | None = None, row_sigmas=None) -> LogitInputs:
    """Draft logits ~N(0, sigma_draft^2), target = draft + N(0, sigma_noise^2).

    Rows follow cu_q / cu_d (packed or padded); rows a sequence does not use
    are still filled.  Draft tokens are exact draws from softmax(draft/T) by
    the Gumbel-max construction (argmax of draft/T + Gumbel noise) for T > 0
    and the plain argmax for T == 0.  With row_sigmas = (sigma_draft [n_q],
    sigma_noise [n_q]) every target row (and the draft row of the same
    position) has its own two standard deviations (see mixture_rows).
    """
    V = cfg.vocab
    sig = cfg.sigma_noise if sigma_noise is None else sigma_noise
    T = cfg.temperature if temperature is None else temperature
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    if row_sigmas is None:
        base = normal_f32(cfg.seed, _T_BASE, n_q * V, cfg.sigma_draft, step).reshape(n_q, V)
        noise = normal_f32(cfg.seed, _T_NOISE, n_q * V, sig, step).reshape(n_q, V)
    else:
        sd, sn = row_sigmas
        base = normal_f32(cfg.seed, _T_BASE, n_q * V, 1.0, step).reshape(n_q, V) * np.asarray(sd, np.float32)[:, None]
        noise = normal_f32(cfg.seed, _T_NOISE, n_q * V, 1.0, step).reshape(n_q, V) * np.asarray(sn, np.float32)[:, None]
    target = base + noise
    draft = np.empty((max(n_d, 1), V), np.float32)[:n_d]
    for b in range(len(gamma)):
        w = int(cu_d[b + 1] - cu_d[b])          # slab width (gamma_b, or gamma_max if padded)
        draft[cu_d[b]:cu_d[b] + w] = base[cu_q[b]:cu_q[b] + w]
    tokens = np.empty(n_d, np.int32)
    if T > 0:
        rows_per = max(1, (1 << 24) // V)
        for lo in range(0, n_d, rows_per):
            hi = min(n_d, lo + rows_per)
            e = _rng(cfg.seed, _T_GUMBEL, lo, step).standard_exponential((hi - lo, V))
            with np.errstate(divide="ignore"):
                gumbel = -np.log(e)
            tokens[lo:hi] = np.argmax(draft[lo:hi].astype(np.float64) / T + gumbel, axis=1)
    else:
        tokens[:] = np.argmax(draft, axis=1)
    return LogitInputs(target, draft, tokens,
                       uniform_f32(cfg.seed, _T_UACC, n_d, step),
                       uniform_f32(cfg.seed, _T_USAMP, len(gamma), step))


def algorithmic_bytes(cfg: VerifyConfig, seq_len: np.ndarray, gamma: np.ndarray):
    """Bytes the step has to move once: (attention, accept) per step.

    attention: every K and V element of every sequence once, plus Q in and O out;
    accept: every target and draft logit once (greedy sequences need target rows only).
    """
    kv = int(seq_len.astype(np.int64).sum()) * cfg.hkv * cfg.head_dim * 2 * 2
    rows = int((gamma + 1).sum())
    qo = 2 * rows * cfg.hq * cfg.head_dim * 2
    if cfg.temperature > 0:
        acc = (2 * int(gamma.sum()) + cfg.batch) * cfg.vocab * 4
    else:
        acc = rows * cfg.vocab * 4
    return kv + qo, acc
