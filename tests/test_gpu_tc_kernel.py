"""GPU parity of the alternative split-K decode kernel (tcgen05.mma with the unpacked codes in tensor memory,
selected with okq_decode_select(0)) against the oracle: the cases that exercise its super-window pipeline, its flush
points (every eight super-windows, a score above the reference maximum, end of a (sequence, head)), windows that mix
modalities, ragged pieces of fewer than four windows, many short units per CTA and the captioning schedule."""
import numpy as np
import pytest
import torch

from paper_2609_11582_b200 import binding as B
from paper_2609_11582_b200 import workloads as WL
from tests import harness as Hn

pytestmark = pytest.mark.gpu
D, W = 128, 32


@pytest.fixture(autouse=True)
def _tcgen05_kernel():
    prev = B.decode_select(0)
    yield
    B.decode_select(prev)


@pytest.mark.parametrize("splits", [1, 2, 7, 0])
def test_tiny_every_split(splits):
    """One (sequence, head) of 64 windows: 1 CTA (16 super-windows, two periodic flushes), 2, 7 (ragged pieces) and
    one window or less per CTA."""
    c = Hn.Case(WL.WORKLOADS["tiny"])
    ref, _ = c.oracle_attention(0)
    got = c.gpu_decode(0, num_splits=splits)[0]
    print("tcgen05 kernel, splits", splits, Hn.assert_attention_close(got, ref))
    assert c.cache.device_status() == 0


def test_ragged_two_sequences():
    c = Hn.Case(WL.scaled(WL.WORKLOADS["layer7b"], batch=2), n_tokens=2048 + 19)
    ref, _ = c.oracle_attention(0)
    for splits in (0, 1):
        Hn.assert_attention_close(c.gpu_decode(0, num_splits=splits)[0], ref)


def test_every_window_holds_all_three_modalities():
    w = WL.scaled(WL.WORKLOADS["layer7b"], batch=2)
    n = 1024 + 13
    g = torch.Generator().manual_seed(99)
    mod = torch.randint(0, 3, (n,), generator=g, dtype=torch.uint8)
    mod[::97] = 7
    c = Hn.Case(w, n_tokens=n, modality=mod)
    ref, _ = c.oracle_attention(0)
    for splits in (0, 1):
        print("mixed windows:", Hn.assert_attention_close(c.gpu_decode(0, num_splits=splits)[0], ref))


def test_one_modality_long_ranges():
    """2048 windows of one modality in a single CTA per (sequence, head): the accumulation chains in tensor memory
    are cut every eight super-windows; the worst head must stay well inside the tolerance."""
    w = WL.scaled(WL.WORKLOADS["layer7b"], n_tokens=65536 + 3)
    c = Hn.Case(w, modality=torch.zeros(w.n_tokens, dtype=torch.uint8))
    ref, _ = c.oracle_attention(0)
    for splits in (1, 0):
        errs = Hn.assert_attention_close(c.gpu_decode(0, num_splits=splits)[0], ref)
        assert errs[1] < 6e-4, errs
        print("one modality, splits", splits, errs)


def test_growing_scores_force_early_flushes():
    """Keys whose norm grows along the sequence: scores keep exceeding the reference maximum by more than the allowed
    2^8, so the kernel must flush and move its reference many times inside one (sequence, head)."""
    w = WL.scaled(WL.WORKLOADS["tiny"], n_tokens=2048, n_chunks=0)
    c = Hn.Case(w)
    # rebuild layer 0 with keys aligned to the first query head and growing: score of token i ~ 0.04 i
    q0 = c.q[0][0, 0].float()
    n = w.n_tokens
    ramp = torch.linspace(0.0, 1.0, n).view(1, 1, n, 1)
    k = (c.k[0].float() * 0.25 + ramp * 8.0 * (q0 / q0.norm()).view(1, 1, 1, D) * 11.3).to(torch.float16)
    c.k[0] = k
    B.quantize_keys(c.cache, 0, k.cuda(), c.d_signs[0])
    torch.cuda.synchronize()
    ref, _ = c.oracle_attention(0)
    for splits in (1, 2):
        print("growing scores:", Hn.assert_attention_close(c.gpu_decode(0, num_splits=splits)[0], ref))


def test_many_short_units_per_cta():
    w = WL.Workload("short", 5, 8, 128, 16, 8, 64 + 5, 16, 20, 12, 0)
    c = Hn.Case(w)
    got = c.gpu_decode(0, layer_count=w.n_layers)
    for l in range(w.n_layers):
        ref, _ = c.oracle_attention(l)
        Hn.assert_attention_close(got[l], ref)
    assert c.cache.device_status() == 0


def test_matches_the_default_kernel_on_a_middle_sized_grid():
    w = WL.scaled(WL.WORKLOADS["step7b"], n_layers=8, n_tokens=1024 + 7)
    c = Hn.Case(w)
    got = c.gpu_decode(0, layer_count=w.n_layers)
    B.decode_select(1)
    other = c.gpu_decode(0, layer_count=w.n_layers)
    B.decode_select(0)
    assert np.abs(got - other).max() < 1e-3
    for l in (0, 7):
        ref, _ = c.oracle_attention(l)
        Hn.assert_attention_close(got[l], ref)
