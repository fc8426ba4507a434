"""spec_verify_noalloc: the entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not an option -- inside a server whose
memory pool has already claimed the whole GPU, inside a host application's callback that
forbids allocation, or in a decode loop that cannot tolerate the synchronisation an
allocation may bring.  They cannot supply spec_verify's workspace, so the library carries a
fixed 4 MiB scratch array in its device image and this entry point uses it.

The array is shared by all calls and keeps the previous call's contents, so the test makes
calls in a row on DIFFERENT batches (of different size, dtype and kernel set, so stale words
from one would sit exactly where the next reads) and requires each to give what the ordinary
entry point gives on the same inputs.  Both entry points run the same kernels on the same
batch (same automatic choice of the kernel set), so lengths, tokens and status are identical
and the probabilities agree far inside the 1e-5 relative tolerance of the parity tests; the
results are also held against the fp64 oracle under the usual margin rule.  It is kept
in a file that sorts last so that a run stopping at the first failure has already run
every other test; it passes alone in a fresh process as well as after the others.
"""
import ctypes

import numpy as np
import pytest
import torch

from gpu_utils import PROB_RTOL, DeviceBatch, assert_parity
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _noalloc(dev: DeviceBatch):
    """Run the no-allocation entry point through the C ABI into fresh output tensors."""
    w = dev.w
    acc = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
    em = torch.full((w.n_draft_total + w.B,), -9, dtype=torch.int32, device="cuda")
    st = torch.full((w.B,), -9, dtype=torch.int32, device="cuda")
    dp = torch.full((w.n_draft_total,), float("nan"), dtype=torch.float32, device="cuda")
    dq = torch.full((w.n_draft_total,), float("nan"), dtype=torch.float32, device="cuda")
    binding.spec_verify_noalloc(dev.target, dev.draft, dev.tokens, dev.k, dev.temperature, dev.uniforms,
                                acc, em, row_status=st, diag_p_tok=dp, diag_q_tok=dq)
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in (acc, em, st, dp, dq)]


def _same(got, ref):
    for g, r in zip(got[:3], ref[:3]):
        assert np.array_equal(g, r)
    np.testing.assert_allclose(got[3], ref[3], rtol=PROB_RTOL, atol=1e-37)
    np.testing.assert_allclose(got[4], ref[4], rtol=PROB_RTOL, atol=1e-37)


def test_calls_in_a_row_match_the_workspace_entry_point():
    binding.set_path(binding.PATH_AUTO)
    first = DeviceBatch(W.make_config(5, B=48, V=20000))      # bf16, ragged lookahead: ring kernels
    second = DeviceBatch(W.make_config(1, B=3, V=4099))       # fp32, few odd rows: streaming kernels
    ref_first = first.run()
    assert binding.last_path() == binding.PATH_RING
    ref_second = second.run()
    assert binding.last_path() == binding.PATH_STREAMING
    got = _noalloc(first)
    assert binding.last_path() == binding.PATH_RING           # the same kernel set as spec_verify chose
    _same(got, ref_first)
    assert_parity(first.w, got)
    got = _noalloc(second)                                    # reuses the scratch the ring kernels left dirty
    assert binding.last_path() == binding.PATH_STREAMING
    _same(got, ref_second)
    assert_parity(second.w, got)
    _same(_noalloc(first), ref_first)                          # and back again


def test_the_largest_benchmark_shape_fits_the_built_in_scratch():
    """512 ragged sequences over a vocabulary of 128256 need 2.3 MiB of the 4 MiB."""
    assert 0 < binding.workspace_bytes(512, 4400, 128256) <= binding.NOALLOC_SCRATCH_BYTES


def test_batches_beyond_the_built_in_scratch_are_refused():
    B, K, V = 30000, 10, 8
    assert binding.workspace_bytes(B, B * K, V) > binding.NOALLOC_SCRATCH_BYTES
    tl = torch.zeros((B * K + B, V), dtype=torch.float32, device="cuda")
    dl = torch.zeros((B * K, V), dtype=torch.float32, device="cuda")
    tok = torch.zeros(B * K, dtype=torch.int32, device="cuda")
    T = torch.ones(1, dtype=torch.float32, device="cuda")
    u = torch.zeros(B * K + B, dtype=torch.float32, device="cuda")
    acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    em = torch.full((B * K + B,), -9, dtype=torch.int32, device="cuda")
    before = binding.launch_count()
    with pytest.raises(binding.SpecVerifyError) as err:
        binding.spec_verify_noalloc(tl, dl, tok, None, T, u, acc, em, k_uniform=K)
    assert err.value.status == 8 and "built-in" in str(err.value)
    assert binding.launch_count() == before                    # refused before any launch
    torch.cuda.synchronize()
    assert int(acc[0]) == -9
    # the same batch is fine through the ordinary entry point with a caller-owned workspace
    binding.spec_verify(tl, dl, tok, None, T, u, k_uniform=K, accepted_len=acc, emitted_tokens=em)
    torch.cuda.synchronize()
    assert int(acc.min()) >= 0
