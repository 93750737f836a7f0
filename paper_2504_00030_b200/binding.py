"""ctypes binding of libspecverify.so -- argument marshalling only.

Every function here has the name and the arguments of the C entry point it
calls (``include/specverify.h``); torch tensors stand in for device pointers.
Nothing is computed in Python, and there is no fallback: if the shared library
has not been built the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspecverify.so")

SV_OK, SV_EINVAL, SV_EUNSUPPORTED, SV_EALIGN, SV_ECUDA, SV_EWORKSPACE = 0, -1, -2, -3, -4, -5
SV_DEV_BAD_GAMMA, SV_DEV_BAD_PAGE, SV_DEV_BAD_TOKEN = 1, 2, 4
SV_DEV_NONFINITE, SV_DEV_TIMEOUT, SV_DEV_BAD_LEN = 8, 16, 32
SV_GT_FIXED, SV_GT_PROPOSED, SV_GT_LITERAL = 0, 1, 2

EXPORTS = (
    "sv_status_str", "sv_launch_count", "spec_kv_pool_register", "spec_kv_pool_release",
    "spec_verify_attn_workspace_bytes", "spec_verify_attn", "spec_accept_sample_workspace_bytes",
    "spec_accept_sample", "spec_accept_sample_static", "gamma_tune_update", "gamma_tune_init",
    "spec_verify_step_host", "spec_draft_stop_workspace_bytes", "spec_draft_stop", "spec_kv_append",
    "sv_selftest_wait_expiry", "spec_verify_attn_layers", "spec_draft_step_workspace_bytes", "spec_draft_step",
)


class SpecVerifyError(RuntimeError):
    def __init__(self, where: str, status: int):
        self.status = status
        super().__init__(f"{where}: {status_str(status)} ({status})")


class AttnParams(C.Structure):
    _fields_ = [("q", C.c_void_p), ("o", C.c_void_p), ("lse", C.c_void_p), ("pool", C.c_void_p),
                ("block_table", C.c_void_p), ("block_table_stride", C.c_int64),
                ("seq_len", C.c_void_p), ("gamma", C.c_void_p), ("cu_q", C.c_void_p),
                ("batch", C.c_int32), ("gamma_max", C.c_int32), ("hq", C.c_int32),
                ("hkv", C.c_int32), ("head_dim", C.c_int32), ("max_seq_len", C.c_int32),
                ("sm_scale", C.c_float), ("device_status", C.c_void_p)]


class AttnLayersParams(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("pools", C.POINTER(C.c_void_p)), ("q", C.POINTER(C.c_void_p)),
                ("o", C.POINTER(C.c_void_p)), ("lse", C.POINTER(C.c_void_p)), ("k_new", C.POINTER(C.c_void_p)),
                ("v_new", C.POINTER(C.c_void_p)), ("shared", AttnParams)]


class KvAppendParams(C.Structure):
    _fields_ = [("k_new", C.c_void_p), ("v_new", C.c_void_p), ("pool", C.c_void_p),
                ("block_table", C.c_void_p), ("block_table_stride", C.c_int64),
                ("seq_len", C.c_void_p), ("gamma", C.c_void_p), ("cu_q", C.c_void_p),
                ("batch", C.c_int32), ("gamma_max", C.c_int32), ("device_status", C.c_void_p)]


class AcceptParams(C.Structure):
    _fields_ = [("target_logits", C.c_void_p), ("draft_logits", C.c_void_p),
                ("row_stride", C.c_int64), ("vocab", C.c_int32), ("draft_tokens", C.c_void_p),
                ("u_accept", C.c_void_p), ("u_sample", C.c_void_p), ("temperature", C.c_float),
                ("temperature_per_seq", C.c_void_p), ("gamma", C.c_void_p), ("cu_q", C.c_void_p),
                ("cu_d", C.c_void_p), ("batch", C.c_int32), ("gamma_max", C.c_int32),
                ("n_accepted", C.c_void_p), ("out_tokens", C.c_void_p), ("ratio", C.c_void_p),
                ("logZ_p", C.c_void_p), ("logZ_q", C.c_void_p), ("flag_count", C.c_void_p),
                ("device_status", C.c_void_p), ("logits_bf16", C.c_int32)]


class GammaConfigC(C.Structure):
    _fields_ = [("eta", C.c_double), ("delta", C.c_double), ("gamma_min", C.c_int32),
                ("gamma_max", C.c_int32), ("mode", C.c_int32), ("padded_rows", C.c_int32)]


class GammaParams(C.Structure):
    _fields_ = [("n_accepted", C.c_void_p), ("gamma_bar", C.c_void_p), ("gamma", C.c_void_p),
                ("seq_len", C.c_void_p), ("cu_q", C.c_void_p), ("cu_d", C.c_void_p),
                ("batch", C.c_int32), ("config", GammaConfigC), ("trajectory", C.c_void_p),
                ("accepted_log", C.c_void_p), ("step", C.c_int32), ("device_status", C.c_void_p),
                ("n_drafted", C.c_void_p)]


class DraftStopParams(C.Structure):
    _fields_ = [("draft_logits", C.c_void_p), ("row_stride", C.c_int64), ("vocab", C.c_int32),
                ("temperature", C.c_float), ("temperature_per_seq", C.c_void_p), ("tau", C.c_float),
                ("gamma", C.c_void_p), ("cu_d", C.c_void_p), ("batch", C.c_int32), ("gamma_max", C.c_int32),
                ("n_drafted", C.c_void_p), ("top_prob", C.c_void_p), ("device_status", C.c_void_p),
                ("logits_bf16", C.c_int32)]


class DraftStepParams(C.Structure):
    _fields_ = [("draft_logits", C.c_void_p), ("row_stride", C.c_int64), ("vocab", C.c_int32),
                ("temperature", C.c_float), ("temperature_per_seq", C.c_void_p), ("tau", C.c_float),
                ("u_sample", C.c_void_p), ("gamma", C.c_void_p), ("cu_d", C.c_void_p), ("batch", C.c_int32),
                ("gamma_max", C.c_int32), ("n_drafted", C.c_void_p), ("active", C.c_void_p),
                ("draft_tokens", C.c_void_p), ("top_prob", C.c_void_p), ("device_status", C.c_void_p),
                ("logits_bf16", C.c_int32)]


class StepHostIO(C.Structure):
    _fields_ = [("q_host", C.c_void_p), ("target_logits_host", C.c_void_p),
                ("draft_logits_host", C.c_void_p), ("draft_tokens_host", C.c_void_p),
                ("u_accept_host", C.c_void_p), ("u_sample_host", C.c_void_p),
                ("n_q_rows", C.c_int64), ("n_d_rows", C.c_int64), ("n_accepted_host", C.c_void_p),
                ("out_tokens_host", C.c_void_p), ("gamma_next_host", C.c_void_p),
                ("o_host", C.c_void_p)]


_lib = None


def load():
    """Load libspecverify.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2504_00030_b200.build` "
                "(there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        lib.sv_status_str.restype = C.c_char_p
        lib.sv_status_str.argtypes = [C.c_int32]
        lib.sv_launch_count.restype = C.c_uint64
        lib.spec_kv_pool_register.restype = C.c_int32
        lib.spec_kv_pool_register.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                                              C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_void_p)]
        lib.spec_kv_pool_release.restype = C.c_int32
        lib.spec_kv_pool_release.argtypes = [C.c_void_p]
        lib.spec_verify_attn_workspace_bytes.restype = C.c_size_t
        lib.spec_verify_attn_workspace_bytes.argtypes = [C.c_int32] * 6
        lib.spec_accept_sample_workspace_bytes.restype = C.c_size_t
        lib.spec_accept_sample_workspace_bytes.argtypes = [C.c_int32] * 3
        lib.spec_verify_attn.restype = C.c_int32
        lib.spec_verify_attn.argtypes = [C.POINTER(AttnParams), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.spec_accept_sample.restype = C.c_int32
        lib.spec_accept_sample.argtypes = [C.POINTER(AcceptParams), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.spec_accept_sample_static.restype = C.c_int32
        lib.spec_accept_sample_static.argtypes = [C.POINTER(AcceptParams), C.c_void_p]
        lib.gamma_tune_update.restype = C.c_int32
        lib.gamma_tune_update.argtypes = [C.POINTER(GammaParams), C.c_void_p]
        lib.gamma_tune_init.restype = C.c_int32
        lib.gamma_tune_init.argtypes = [C.POINTER(GammaParams), C.c_int32, C.c_void_p]
        lib.spec_verify_attn_layers.restype = C.c_int32
        lib.spec_verify_attn_layers.argtypes = [C.POINTER(AttnLayersParams), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.sv_selftest_wait_expiry.restype = C.c_int32
        lib.sv_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        lib.spec_draft_stop_workspace_bytes.restype = C.c_size_t
        lib.spec_draft_stop_workspace_bytes.argtypes = [C.c_int32] * 3
        lib.spec_draft_stop.restype = C.c_int32
        lib.spec_draft_stop.argtypes = [C.POINTER(DraftStopParams), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.spec_draft_step_workspace_bytes.restype = C.c_size_t
        lib.spec_draft_step_workspace_bytes.argtypes = [C.c_int32] * 2
        lib.spec_draft_step.restype = C.c_int32
        lib.spec_draft_step.argtypes = [C.POINTER(DraftStepParams), C.c_void_p, C.c_size_t, C.c_void_p]
        lib.spec_verify_step_host.restype = C.c_int32
        lib.spec_verify_step_host.argtypes = [C.POINTER(StepHostIO), C.POINTER(AttnParams), C.c_void_p,
                                              C.c_size_t, C.POINTER(AcceptParams), C.c_void_p,
                                              C.c_size_t, C.POINTER(GammaParams), C.c_void_p]
        _lib = lib
    return _lib


def status_str(status: int) -> str:
    return load().sv_status_str(int(status)).decode()


def sv_launch_count() -> int:
    return int(load().sv_launch_count())


def _check(where: str, status: int):
    if status != SV_OK:
        raise SpecVerifyError(where, status)


def _dev(t, dtype, name, allow_none=False):
    """Device pointer of a CUDA tensor (dtype and contiguity checked)."""
    if t is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _dev_rows(t, dtype, name):
    """Device pointer of a 2-D CUDA tensor whose rows are contiguous; the rows may be strided."""
    if t is None or not t.is_cuda or t.dtype != dtype or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name} must be a 2-D CUDA tensor of {dtype} with contiguous rows")
    return t.data_ptr()


def _host(t, dtype, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise ValueError(f"{name} is required")
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor of {dtype}")
    return t.data_ptr()


def _nbytes(t) -> int:
    return t.numel() * t.element_size()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


# --------------------------------------------------------------------------- KV pool
class KVPool:
    """Handle of a registered paged KV pool (keeps the tensors alive)."""

    def __init__(self, k_pool: torch.Tensor, v_pool: torch.Tensor, strides=None):
        if k_pool.dim() != 4 or k_pool.shape != v_pool.shape:
            raise ValueError("pools must be 4-D [n_pages, hkv, page_size, head_dim] and alike")
        n_pages, hkv, page_size, head_dim = k_pool.shape
        if strides is None:
            strides = k_pool.stride()
            if tuple(v_pool.stride()) != tuple(strides):
                raise ValueError("K and V pools must share their strides")
        if not (k_pool.is_cuda and v_pool.is_cuda and k_pool.dtype == torch.bfloat16 and
                v_pool.dtype == torch.bfloat16):
            raise ValueError("pools must be CUDA bf16 tensors")
        self.k_pool, self.v_pool = k_pool, v_pool
        self.n_pages, self.hkv, self.page_size, self.head_dim = n_pages, hkv, page_size, head_dim
        st = (C.c_int64 * 4)(*[int(s) for s in strides])
        handle = C.c_void_p()
        self.handle = None
        _check("spec_kv_pool_register",
               load().spec_kv_pool_register(k_pool.data_ptr(), v_pool.data_ptr(), n_pages, page_size,
                                            hkv, head_dim, st, C.byref(handle)))
        self.handle = handle

    def release(self):
        if self.handle is not None and self.handle.value:
            load().spec_kv_pool_release(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.release()
        except Exception:
            pass


def spec_kv_pool_register(k_pool, v_pool, strides=None) -> KVPool:
    return KVPool(k_pool, v_pool, strides)


# --------------------------------------------------------------------------- attention
def spec_verify_attn_workspace_bytes(batch, gamma_max, hq, hkv, head_dim, max_seq_len) -> int:
    return int(load().spec_verify_attn_workspace_bytes(batch, gamma_max, hq, hkv, head_dim, max_seq_len))


def attn_params(q, o, pool: KVPool, block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len,
                sm_scale=None, lse=None, device_status=None) -> AttnParams:
    n_rows, hq, head_dim = q.shape
    p = AttnParams()
    p.q = _dev(q, torch.bfloat16, "q")
    p.o = _dev(o, torch.bfloat16, "o")
    p.lse = _dev(lse, torch.float32, "lse", True)
    p.pool = pool.handle
    p.block_table = _dev(block_table, torch.int32, "block_table")
    p.block_table_stride = block_table.shape[1]
    p.seq_len = _dev(seq_len, torch.int32, "seq_len")
    p.gamma = _dev(gamma, torch.int32, "gamma")
    p.cu_q = _dev(cu_q, torch.int32, "cu_q")
    p.batch = seq_len.shape[0]
    p.gamma_max = gamma_max
    p.hq, p.hkv, p.head_dim = hq, pool.hkv, head_dim
    p.max_seq_len = max_seq_len
    p.sm_scale = float(sm_scale) if sm_scale is not None else head_dim ** -0.5
    p.device_status = _dev(device_status, torch.int32, "device_status", True)
    return p


def spec_verify_attn(q, o, pool, block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len,
                     workspace, sm_scale=None, lse=None, device_status=None, stream=None):
    """Attention of the draft block against the paged KV cache (asynchronous)."""
    p = attn_params(q, o, pool, block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len,
                    sm_scale, lse, device_status)
    _check("spec_verify_attn",
           load().spec_verify_attn(C.byref(p), workspace.data_ptr(), _nbytes(workspace), _stream(stream)))


def kv_append_params(k_new, v_new, pool, block_table, seq_len, gamma, cu_q, gamma_max,
                     device_status=None) -> KvAppendParams:
    p = KvAppendParams()
    p.k_new = _dev(k_new, torch.bfloat16, "k_new")
    p.v_new = _dev(v_new, torch.bfloat16, "v_new")
    if tuple(k_new.shape) != tuple(v_new.shape) or k_new.dim() != 3:
        raise ValueError("k_new and v_new must both be [n_rows, hkv, head_dim]")
    if tuple(k_new.shape[1:]) != (pool.hkv, pool.head_dim):
        raise ValueError("k_new rows do not match the pool's heads and head_dim")
    p.pool = pool.handle
    p.block_table = _dev(block_table, torch.int32, "block_table")
    p.block_table_stride = block_table.shape[1]
    p.seq_len = _dev(seq_len, torch.int32, "seq_len")
    p.gamma = _dev(gamma, torch.int32, "gamma")
    p.cu_q = _dev(cu_q, torch.int32, "cu_q")
    p.batch = gamma.shape[0]
    p.gamma_max = gamma_max
    p.device_status = _dev(device_status, torch.int32, "device_status", True)
    return p


def spec_kv_append(k_new, v_new, pool, block_table, seq_len, gamma, cu_q, gamma_max, device_status=None,
                   stream=None):
    """Write the draft block's keys and values behind each sequence's context (asynchronous)."""
    p = kv_append_params(k_new, v_new, pool, block_table, seq_len, gamma, cu_q, gamma_max, device_status)
    _check("spec_kv_append", load().spec_kv_append(C.byref(p), _stream(stream)))


# --------------------------------------------------------------------------- accept / resample
def spec_accept_sample_workspace_bytes(batch, gamma_max, vocab) -> int:
    return int(load().spec_accept_sample_workspace_bytes(batch, gamma_max, vocab))


def accept_params(target_logits, draft_logits, draft_tokens, u_accept, u_sample, temperature, gamma,
                  cu_q, cu_d, gamma_max, n_accepted, out_tokens, ratio=None, logZ_p=None,
                  logZ_q=None, flag_count=None, device_status=None,
                  temperature_per_seq=None) -> AcceptParams:
    p = AcceptParams()
    ldt = target_logits.dtype if target_logits.dtype == torch.bfloat16 else torch.float32     # float32 or bf16 logits
    p.logits_bf16 = int(ldt == torch.bfloat16)
    p.target_logits = _dev(target_logits, ldt, "target_logits")
    p.draft_logits = _dev(draft_logits, ldt, "draft_logits", True)
    p.row_stride = target_logits.stride(0)
    p.vocab = target_logits.shape[-1]
    p.draft_tokens = _dev(draft_tokens, torch.int32, "draft_tokens", True)
    p.u_accept = _dev(u_accept, torch.float32, "u_accept", True)
    p.u_sample = _dev(u_sample, torch.float32, "u_sample", True)
    p.temperature = float(temperature)
    p.temperature_per_seq = _dev(temperature_per_seq, torch.float32, "temperature_per_seq", True)
    p.gamma = _dev(gamma, torch.int32, "gamma")
    p.cu_q = _dev(cu_q, torch.int32, "cu_q")
    p.cu_d = _dev(cu_d, torch.int32, "cu_d")
    p.batch = gamma.shape[0]
    p.gamma_max = gamma_max
    p.n_accepted = _dev(n_accepted, torch.int32, "n_accepted")
    p.out_tokens = _dev(out_tokens, torch.int32, "out_tokens")
    p.ratio = _dev(ratio, torch.float64, "ratio", True)
    p.logZ_p = _dev(logZ_p, torch.float64, "logZ_p", True)
    p.logZ_q = _dev(logZ_q, torch.float64, "logZ_q", True)
    p.flag_count = _dev(flag_count, torch.int32, "flag_count", True)
    p.device_status = _dev(device_status, torch.int32, "device_status", True)
    return p


def spec_accept_sample(target_logits, draft_logits, draft_tokens, u_accept, u_sample, temperature,
                       gamma, cu_q, cu_d, gamma_max, n_accepted, out_tokens, workspace, ratio=None,
                       logZ_p=None, logZ_q=None, flag_count=None, device_status=None,
                       temperature_per_seq=None, stream=None):
    """Accept / reject the drafts and draw the next token (asynchronous)."""
    p = accept_params(target_logits, draft_logits, draft_tokens, u_accept, u_sample, temperature,
                      gamma, cu_q, cu_d, gamma_max, n_accepted, out_tokens, ratio, logZ_p, logZ_q,
                      flag_count, device_status, temperature_per_seq)
    _check("spec_accept_sample",
           load().spec_accept_sample(C.byref(p), workspace.data_ptr(), _nbytes(workspace),
                                     _stream(stream)))


SV_ACCEPT_STATIC_SCRATCH_BYTES = 8 << 20


def spec_accept_sample_static(target_logits, draft_logits, draft_tokens, u_accept, u_sample, temperature,
                              gamma, cu_q, cu_d, gamma_max, n_accepted, out_tokens, ratio=None,
                              logZ_p=None, logZ_q=None, flag_count=None, device_status=None,
                              temperature_per_seq=None, stream=None):
    """spec_accept_sample for callers that cannot hand over scratch memory (no workspace
    argument; the library's built-in array is used).  Problems beyond that array's size raise
    SpecVerifyError with SV_EWORKSPACE.  Calls on one device must not overlap on the GPU."""
    p = accept_params(target_logits, draft_logits, draft_tokens, u_accept, u_sample, temperature,
                      gamma, cu_q, cu_d, gamma_max, n_accepted, out_tokens, ratio, logZ_p, logZ_q,
                      flag_count, device_status, temperature_per_seq)
    _check("spec_accept_sample_static", load().spec_accept_sample_static(C.byref(p), _stream(stream)))


# --------------------------------------------------------------------------- GammaTune
@dataclass
class GammaConfig:
    eta: float = 0.5
    delta: float = 2.0
    gamma_min: int = 1
    gamma_max: int = 8
    mode: int = SV_GT_PROPOSED
    padded_rows: bool = False


def gamma_params(n_accepted, gamma_bar, gamma, seq_len, cu_q, cu_d, config: GammaConfig,
                 trajectory=None, accepted_log=None, step=0, device_status=None, n_drafted=None) -> GammaParams:
    p = GammaParams()
    p.n_accepted = _dev(n_accepted, torch.int32, "n_accepted", True)
    p.gamma_bar = _dev(gamma_bar, torch.float64, "gamma_bar")
    p.gamma = _dev(gamma, torch.int32, "gamma")
    p.seq_len = _dev(seq_len, torch.int32, "seq_len", True)
    p.cu_q = _dev(cu_q, torch.int32, "cu_q")
    p.cu_d = _dev(cu_d, torch.int32, "cu_d")
    p.batch = gamma.shape[0]
    p.config = GammaConfigC(config.eta, config.delta, config.gamma_min, config.gamma_max,
                            config.mode, int(config.padded_rows))
    p.trajectory = _dev(trajectory, torch.int32, "trajectory", True)
    p.accepted_log = _dev(accepted_log, torch.int32, "accepted_log", True)
    p.step = step
    p.device_status = _dev(device_status, torch.int32, "device_status", True)
    p.n_drafted = _dev(n_drafted, torch.int32, "n_drafted", True)
    return p


def gamma_tune_update(n_accepted, gamma_bar, gamma, seq_len, cu_q, cu_d, config: GammaConfig,
                      trajectory=None, accepted_log=None, step=0, device_status=None, stream=None,
                      n_drafted=None):
    """One GammaTune update of every sequence's (gamma_bar, gamma) on the device (asynchronous)."""
    p = gamma_params(n_accepted, gamma_bar, gamma, seq_len, cu_q, cu_d, config, trajectory,
                     accepted_log, step, device_status, n_drafted)
    _check("gamma_tune_update", load().gamma_tune_update(C.byref(p), _stream(stream)))


# --------------------------------------------------------------------------- GammaTune+ early stop
def spec_draft_stop_workspace_bytes(batch, gamma_max, vocab) -> int:
    return int(load().spec_draft_stop_workspace_bytes(batch, gamma_max, vocab))


def draft_stop_params(draft_logits, temperature, tau, gamma, cu_d, gamma_max, n_drafted, top_prob=None,
                      device_status=None, temperature_per_seq=None) -> DraftStopParams:
    p = DraftStopParams()
    ldt = draft_logits.dtype if draft_logits.dtype == torch.bfloat16 else torch.float32       # float32 or bf16 logits
    p.logits_bf16 = int(ldt == torch.bfloat16)
    p.draft_logits = _dev(draft_logits, ldt, "draft_logits")
    p.row_stride = draft_logits.stride(0)
    p.vocab = draft_logits.shape[-1]
    p.temperature = float(temperature)
    p.temperature_per_seq = _dev(temperature_per_seq, torch.float32, "temperature_per_seq", True)
    p.tau = float(tau)
    p.gamma = _dev(gamma, torch.int32, "gamma")
    p.cu_d = _dev(cu_d, torch.int32, "cu_d")
    p.batch = gamma.shape[0]
    p.gamma_max = gamma_max
    p.n_drafted = _dev(n_drafted, torch.int32, "n_drafted")
    p.top_prob = _dev(top_prob, torch.float64, "top_prob", True)
    p.device_status = _dev(device_status, torch.int32, "device_status", True)
    return p


def spec_draft_stop(draft_logits, temperature, tau, gamma, cu_d, gamma_max, n_drafted, workspace,
                    top_prob=None, device_status=None, temperature_per_seq=None, stream=None):
    """GammaTune+ early stop of drafting: n_drafted per sequence (asynchronous)."""
    p = draft_stop_params(draft_logits, temperature, tau, gamma, cu_d, gamma_max, n_drafted, top_prob,
                          device_status, temperature_per_seq)
    _check("spec_draft_stop",
           load().spec_draft_stop(C.byref(p), workspace.data_ptr(), _nbytes(workspace), _stream(stream)))


# --------------------------------------------------------------------------- GammaTune+ drafting step
def spec_draft_step_workspace_bytes(batch, vocab) -> int:
    return int(load().spec_draft_step_workspace_bytes(batch, vocab))


def draft_step_params(draft_logits, temperature, tau, u_sample, gamma, cu_d, gamma_max, n_drafted, active,
                      draft_tokens, top_prob=None, device_status=None, temperature_per_seq=None) -> DraftStepParams:
    p = DraftStepParams()
    ldt = draft_logits.dtype if draft_logits.dtype == torch.bfloat16 else torch.float32       # float32 or bf16 logits
    p.logits_bf16 = int(ldt == torch.bfloat16)
    p.draft_logits = _dev_rows(draft_logits, ldt, "draft_logits")     # e.g. position i of every block
    p.row_stride = draft_logits.stride(0)
    p.vocab = draft_logits.shape[-1]
    p.temperature = float(temperature)
    p.temperature_per_seq = _dev(temperature_per_seq, torch.float32, "temperature_per_seq", True)
    p.tau = float(tau)
    p.u_sample = _dev(u_sample, torch.float32, "u_sample", True)
    p.gamma = _dev(gamma, torch.int32, "gamma")
    p.cu_d = _dev(cu_d, torch.int32, "cu_d")
    p.batch = gamma.shape[0]
    p.gamma_max = gamma_max
    p.n_drafted = _dev(n_drafted, torch.int32, "n_drafted")
    p.active = _dev(active, torch.int32, "active")
    p.draft_tokens = _dev(draft_tokens, torch.int32, "draft_tokens")
    p.top_prob = _dev(top_prob, torch.float64, "top_prob", True)
    p.device_status = _dev(device_status, torch.int32, "device_status", True)
    return p


def spec_draft_step(draft_logits, temperature, tau, u_sample, gamma, cu_d, gamma_max, n_drafted, active,
                    draft_tokens, workspace, top_prob=None, device_status=None, temperature_per_seq=None,
                    stream=None):
    """One drafting step with the confidence stop (asynchronous): token, top probability, n_drafted, active."""
    p = draft_step_params(draft_logits, temperature, tau, u_sample, gamma, cu_d, gamma_max, n_drafted, active,
                          draft_tokens, top_prob, device_status, temperature_per_seq)
    _check("spec_draft_step",
           load().spec_draft_step(C.byref(p), workspace.data_ptr(), _nbytes(workspace), _stream(stream)))


def gamma_tune_init(gamma_bar, gamma, cu_q, cu_d, config: GammaConfig, gamma0: int, stream=None):
    p = gamma_params(None, gamma_bar, gamma, None, cu_q, cu_d, config)
    _check("gamma_tune_init", load().gamma_tune_init(C.byref(p), int(gamma0), _stream(stream)))


# --------------------------------------------------------------------------- step from host buffers
def spec_verify_step_host(io: StepHostIO, attn: AttnParams, attn_workspace, accept: AcceptParams,
                          accept_workspace, gamma: GammaParams, stream=None):
    """One whole verify step whose per-step inputs start in (pinned) host memory."""
    _check("spec_verify_step_host",
           load().spec_verify_step_host(
               C.byref(io), C.byref(attn), attn_workspace.data_ptr(), _nbytes(attn_workspace),
               C.byref(accept), accept_workspace.data_ptr(), _nbytes(accept_workspace),
               C.byref(gamma), _stream(stream)))


def step_host_io(q_host, target_logits_host, draft_logits_host, draft_tokens_host, u_accept_host,
                 u_sample_host, n_q_rows, n_d_rows, n_accepted_host, out_tokens_host,
                 gamma_next_host, o_host=None) -> StepHostIO:
    io = StepHostIO()
    io.q_host = _host(q_host, torch.bfloat16, "q_host")
    io.target_logits_host = _host(target_logits_host, torch.float32, "target_logits_host")
    io.draft_logits_host = _host(draft_logits_host, torch.float32, "draft_logits_host", True)
    io.draft_tokens_host = _host(draft_tokens_host, torch.int32, "draft_tokens_host", True)
    io.u_accept_host = _host(u_accept_host, torch.float32, "u_accept_host", True)
    io.u_sample_host = _host(u_sample_host, torch.float32, "u_sample_host", True)
    io.n_q_rows, io.n_d_rows = int(n_q_rows), int(n_d_rows)
    io.n_accepted_host = _host(n_accepted_host, torch.int32, "n_accepted_host")
    io.out_tokens_host = _host(out_tokens_host, torch.int32, "out_tokens_host")
    io.gamma_next_host = _host(gamma_next_host, torch.int32, "gamma_next_host")
    io.o_host = _host(o_host, torch.bfloat16, "o_host", True)
    return io


# --------------------------------------------------------------------------- all layers of a step
def attn_layers_params(qs, os_, pools, block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len, k_new=None,
                       v_new=None, lses=None, sm_scale=None, device_status=None) -> AttnLayersParams:
    """Arguments of spec_verify_attn_layers: lists with one entry per layer, the rest shared.  The returned
    struct keeps the pointer arrays alive."""
    n = len(pools)
    if not (len(qs) == n and len(os_) == n):
        raise ValueError("one q, o and pool per layer")
    p = AttnLayersParams()
    p.n_layers = n
    p.shared = attn_params(qs[0], os_[0], pools[0], block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len,
                           sm_scale, None, device_status)

    def arr(ptrs):
        a = (C.c_void_p * n)(*ptrs)
        return a

    p._keep = [arr([pl.handle.value for pl in pools]), arr([_dev(t, torch.bfloat16, "q") for t in qs]),
               arr([_dev(t, torch.bfloat16, "o") for t in os_])]
    p.pools, p.q, p.o = (C.cast(a, C.POINTER(C.c_void_p)) for a in p._keep)
    if lses is not None:
        a = arr([_dev(t, torch.float32, "lse") for t in lses])
        p._keep.append(a)
        p.lse = C.cast(a, C.POINTER(C.c_void_p))
    if k_new is not None:
        ak = arr([_dev(t, torch.bfloat16, "k_new") for t in k_new])
        av = arr([_dev(t, torch.bfloat16, "v_new") for t in v_new])
        p._keep += [ak, av]
        p.k_new, p.v_new = C.cast(ak, C.POINTER(C.c_void_p)), C.cast(av, C.POINTER(C.c_void_p))
    return p


def spec_verify_attn_layers(qs, os_, pools, block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len, workspace,
                            k_new=None, v_new=None, lses=None, sm_scale=None, device_status=None, stream=None):
    """Cache append (one launch for all layers) and verify attention of every layer's cache (asynchronous)."""
    p = attn_layers_params(qs, os_, pools, block_table, seq_len, gamma, cu_q, gamma_max, max_seq_len, k_new, v_new,
                           lses, sm_scale, device_status)
    _check("spec_verify_attn_layers",
           load().spec_verify_attn_layers(C.byref(p), workspace.data_ptr(), _nbytes(workspace), _stream(stream)))


# --------------------------------------------------------------------------- self-test
def sv_selftest_wait_expiry(device_status, device_result, limit_cycles, stream=None):
    """One thread block waits, with a budget of `limit_cycles`, on a barrier nothing arrives at."""
    _check("sv_selftest_wait_expiry",
           load().sv_selftest_wait_expiry(_dev(device_status, torch.int32, "device_status"),
                                          _dev(device_result, torch.int32, "device_result"),
                                          int(limit_cycles), _stream(stream)))
