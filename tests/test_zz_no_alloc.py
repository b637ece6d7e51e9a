"""okq_decode_attention_noalloc: the decode call for users who cannot allocate scratch.

Some callers of this library run where device allocation is not allowed at call time: a serving
loop whose memory pool was fixed at start-up, a plugin that only receives its inputs and
outputs.  For them the library carries its own 64 MiB scratch array per GPU.  This test calls
the entry point through the C ABI twice in a row (the array keeps the previous call's contents,
so the second call shows that nothing stale is picked up) and checks each result against
okq_decode_attention with a caller-owned workspace, and against the CPU oracle.

The file sorts last on purpose: a run that stops at the first failure has then already run
every other test.  It also passes on its own in a fresh process.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

D = 128


def test_noalloc_rejects_oversized_request_without_a_gpu():
    # 48 layers x 16 sequences x 4 heads = 3072 partials + the CTAs: more than the 64 MiB scratch holds
    c = B.okq_cache(48, 16, 4, 32, 128, 32, 32768, 0, 0, 0, 1 << 20, 1 << 20, 1 << 20, 1 << 20, 1 << 20, 1 << 20)
    st = B.lib().okq_decode_attention_noalloc(C.byref(c), 0, 48, 1 << 20, 0.1, 1 << 20, 1 << 20, 1, 0, 1 << 20, None)
    assert st == B.ERR_WORKSPACE
    bad = B.okq_cache(1, 1, 1, 7, 64, 32, 64, 0)
    assert B.lib().okq_decode_attention_noalloc(C.byref(bad), 0, 1, 1 << 20, 0.1, 1 << 20, 1 << 20, 1, 0, 1 << 20,
                                                None) == B.ERR_UNSUPPORTED


@pytest.mark.gpu
def test_noalloc_matches_decode_attention_twice_in_a_row():
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2, n_layers=2)
    case = Hn.Case(w, n_tokens=1024 + 13)
    cache, dev = case.cache, case.cache.device
    refs = [case.oracle_attention(l)[0] for l in range(2)]
    want = case.gpu_decode(0, layer_count=2)            # caller-owned workspace
    for call in range(2):
        out = torch.full((2, w.batch, w.n_q_heads, D), float("nan"), dtype=torch.float32, device=dev)
        B.decode_attention_noalloc(cache, 0, 2, case.d_q, case.d_signs, case.d_R, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy().astype(np.float64)
        rel, worst, mx = Hn.attention_errors(got, want)
        assert rel < Hn.REL_L2_TOL and worst < Hn.REL_L2_TOL and mx < Hn.MAX_ABS_TOL, (call, rel, worst, mx)
        for l in range(2):
            Hn.assert_attention_close(got[l], refs[l])
        # a different query between the calls, so that stale partials would show
        case.d_q = torch.flip(case.d_q, dims=[2]).contiguous()
        case.q = torch.flip(case.q, dims=[2]).contiguous()
        refs = [case.oracle_attention(l)[0] for l in range(2)]
        want = case.gpu_decode(0, layer_count=2)
    assert cache.device_status() == 0


@pytest.mark.gpu
@pytest.mark.parametrize("meta_format,num_splits", [(B.META_MXFP4, 0), (B.META_FP16, 3), (B.META_MXFP4, 5)])
def test_noalloc_other_formats_and_grids(meta_format, num_splits):
    """The same comparison with MXFP4 metadata and with a caller-chosen number of CTAs per (sequence, head): both reuse
    the library's scratch with a different partition of it.  Twice in a row, against the caller-owned-workspace call."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=3, n_layers=2)
    case = Hn.Case(w, n_tokens=512 + 9, meta_format=meta_format)
    cache, dev = case.cache, case.cache.device
    for call in range(2):
        want = case.gpu_decode(0, layer_count=2, num_splits=num_splits)
        out = torch.full((2, w.batch, w.n_q_heads, D), float("nan"), dtype=torch.float32, device=dev)
        B.decode_attention_noalloc(cache, 0, 2, case.d_q, case.d_signs, case.d_R, out, num_splits=num_splits)
        torch.cuda.synchronize()
        got = out.cpu().numpy().astype(np.float64)
        rel, worst, mx = Hn.attention_errors(got, want)
        assert rel < Hn.REL_L2_TOL and worst < Hn.REL_L2_TOL and mx < Hn.MAX_ABS_TOL, (call, rel, worst, mx)
        case.d_q = torch.flip(case.d_q, dims=[2]).contiguous()
    assert cache.device_status() == 0
