"""spec_accept_sample_static: the accept / resample step for callers that cannot allocate.

Some users of this library cannot give it scratch memory: an engine whose device memory was
handed out completely at start-up, or a host framework that forbids (or would stall on) a
cudaMalloc at the point of the call.  For them the library carries a fixed scratch array of its
own.  This test calls that entry point through the C ABI, twice in a row on different inputs
(the second call finds the first call's leftovers in the shared array), and checks every output
against the regular entry point; the counts and tokens are compared with the oracle as well.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2504_00030_b200 import binding as sv
from paper_2504_00030_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def run_both(cfg, step):
    """Runs the regular and the no-allocation entry point on the same inputs; returns both outputs."""
    _, gamma = synth.draw_lengths(cfg, step)
    cu_q, cu_d = synth.prefix(gamma)
    li = synth.make_logits(cfg, gamma, cu_q, cu_d, step)
    B, gmax, V = cfg.batch, cfg.gamma_max, cfg.vocab
    n_q, n_d = int(cu_q[-1]), int(cu_d[-1])
    ins = (dev(li.target_logits), dev(li.draft_logits), dev(li.draft_tokens), dev(li.u_accept),
           dev(li.u_sample))
    idx = (dev(gamma), dev(cu_q), dev(cu_d))

    def outputs():
        return dict(n=torch.full((B,), -9, dtype=torch.int32, device=DEV),
                    tok=torch.full((B, gmax + 1), -9, dtype=torch.int32, device=DEV),
                    ratio=torch.full((n_d,), float("nan"), dtype=torch.float64, device=DEV),
                    lzp=torch.full((n_q,), float("nan"), dtype=torch.float64, device=DEV),
                    lzq=torch.full((n_d,), float("nan"), dtype=torch.float64, device=DEV),
                    status=torch.zeros(1, dtype=torch.int32, device=DEV))

    ref, got = outputs(), outputs()
    ws = torch.empty(sv.spec_accept_sample_workspace_bytes(B, gmax, V), dtype=torch.uint8, device=DEV)
    sv.spec_accept_sample(*ins, cfg.temperature, *idx, gmax, ref["n"], ref["tok"], ws, ratio=ref["ratio"],
                          logZ_p=ref["lzp"], logZ_q=ref["lzq"], device_status=ref["status"])
    # the new entry point, straight through the C ABI: parameter struct + stream, nothing else
    p = sv.accept_params(*ins, cfg.temperature, *idx, gmax, got["n"], got["tok"], ratio=got["ratio"],
                         logZ_p=got["lzp"], logZ_q=got["lzq"], device_status=got["status"])
    st = sv.load().spec_accept_sample_static(C.byref(p), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert st == sv.SV_OK, sv.status_str(st)
    torch.cuda.synchronize()
    # and against the oracle directly (counts and token ids, near ties followed as in the other accept tests)
    from tests.harness import AcceptOut, compare_accept
    out = AcceptOut(got["n"].cpu().numpy(), got["tok"].cpu().numpy(), got["ratio"].cpu().numpy(),
                    got["lzp"].cpu().numpy(), got["lzq"].cpu().numpy(), 0, 0)
    compare_accept(out, li, cfg.temperature, gamma, cu_q, cu_d, gmax)
    return ref, got


def assert_same(ref, got):
    assert ref["status"].item() == 0 and got["status"].item() == 0
    # accepted counts and token ids: exact, as everywhere in the accept tests
    assert torch.equal(ref["n"], got["n"])
    assert torch.equal(ref["tok"], got["tok"])
    # softmax sums to the 1e-5 relative bound of the accept tests, ratios to 1e-6
    for key, tol in (("lzp", 1e-5), ("lzq", 1e-5), ("ratio", 1e-6)):
        a, b = ref[key].cpu().numpy(), got[key].cpu().numpy()
        assert np.array_equal(np.isnan(a), np.isnan(b))
        ok = ~np.isnan(a)
        if not ok.any():
            continue
        if key == "ratio":
            assert np.abs(a[ok] - b[ok]).max() <= tol
        else:
            assert np.abs(np.expm1(a[ok] - b[ok])).max() <= tol


def test_two_calls_in_a_row_match_the_regular_entry_point():
    big = synth.scaled(synth.CONFIGS["c3"], batch=12)                 # V = 128256, gamma 2..10
    small = synth.VerifyConfig("small", 5, 1, 1, 64, 4099, 32, 32, 0, 6, 6, 0.8, 0.6, seed=123)
    ref, got = run_both(big, step=0)
    assert_same(ref, got)
    assert (ref["n"] > 0).any() and (ref["tok"][:, 0] >= 0).all()
    # second call, smaller and differently shaped: the array still holds the first call's records
    ref, got = run_both(small, step=1)
    assert_same(ref, got)


def test_problem_larger_than_the_built_in_array_is_refused():
    B, gmax, V = 4096, 16, 128256            # slice statistics alone: 4096 * 33 * 8 * 32 B = 34.6 MB > 8 MiB
    z = torch.zeros(1, dtype=torch.float32, device=DEV)
    i = torch.zeros(1, dtype=torch.int32, device=DEV)
    p = sv.AcceptParams()
    p.target_logits = p.draft_logits = p.u_accept = p.u_sample = z.data_ptr()
    p.draft_tokens = p.gamma = p.cu_q = p.cu_d = p.n_accepted = p.out_tokens = i.data_ptr()
    p.row_stride, p.vocab, p.batch, p.gamma_max, p.temperature = V, V, B, gmax, 1.0
    st = sv.load().spec_accept_sample_static(C.byref(p), None)
    assert st == sv.SV_EWORKSPACE
    assert "workspace" in sv.status_str(st)
