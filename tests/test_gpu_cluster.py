"""The one-launch form for small batches (a thread-block cluster of eight CTAs per sequence holding
the sequence's logits rows in shared memory) against the fp64 oracle, through the C ABI: it must be
the form that runs on the shapes it is meant for, agree with the oracle like the other kernel sets,
and hand batches it cannot hold to them."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import DeviceBatch, assert_parity, run_oracle
from helpers import Case
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _automatic_choice():
    binding.set_path(binding.PATH_AUTO)
    yield
    binding.set_path(binding.PATH_AUTO)


@pytest.mark.parametrize("cfg,B,V,K", [(1, 1, 32000, 4),       # fp32, the single-sequence workload
                                       (2, 8, 32000, 5),       # bf16, the eight-sequence workload
                                       (2, 18, 4096, 3),       # as many sequences as the form takes
                                       (1, 2, 1000, 32),       # the longest lookahead it takes; rows that are not whole segments
                                       (2, 2, 128256, 1),      # a large vocabulary with a short lookahead
                                       (1, 5, 8, 2), (2, 4, 8, 0)])   # tiny rows: most CTAs of a cluster hold nothing; K = 0
@pytest.mark.parametrize("uniform", [True, False])
def test_parity_on_the_shapes_it_takes(cfg, B, V, K, uniform):
    w = W.make_config(cfg, B=B, V=V, K=K)
    dev = DeviceBatch(w)
    got = dev.run(use_k_per_row=not uniform, k_uniform=K if uniform else None)
    # with a per-sequence lookahead array the host cannot see the lookahead: the draft rows bound it
    takes = uniform or w.n_draft_total <= 32
    assert (binding.last_path() == binding.PATH_CLUSTER) == takes
    assert_parity(w, got, max_excused_frac=0.2)


def test_fp16_and_ragged_lookahead():
    w = W.make_config(5, B=16, V=4096)                        # ragged K_b in 1..16
    b1 = 1
    while b1 < w.B and int(w.k_per_row[:b1 + 1].sum()) <= 32:
        b1 += 1
    sub = w.take(0, b1)                                       # as many sequences as keep the draft rows at 32 or fewer
    assert sub.B >= 2 and sub.n_draft_total <= 32
    got = DeviceBatch(sub).run()
    assert binding.last_path() == binding.PATH_CLUSTER
    assert_parity(sub, got, max_excused_frac=0.5)
    h = W.make_config(2, B=6, V=12000, K=4, dtype="f16")
    got = DeviceBatch(h).run(use_k_per_row=False, k_uniform=4)
    assert binding.last_path() == binding.PATH_CLUSTER
    assert_parity(h, got, max_excused_frac=0.2)


def test_batches_it_cannot_hold_go_to_the_other_kernels():
    for w, why in ((W.make_config(2, B=19, V=4096, K=3), "too many sequences"),
                   (W.make_config(2, B=4, V=4096, K=33), "lookahead beyond the tables"),
                   (W.make_config(1, B=2, V=4099, K=2), "rows that are not whole 16-byte vectors"),
                   (W.make_config(1, B=1, V=200000, K=4), "rows beyond a cluster's shared memory")):
        got = DeviceBatch(w).run(use_k_per_row=False, k_uniform=int(w.k_per_row[0]))
        assert binding.last_path() in (binding.PATH_STREAMING, binding.PATH_RING), why
        assert_parity(w, got, max_excused_frac=0.5)
    w = W.make_config(2, B=4, V=4096, K=3)
    DeviceBatch(w, elem_offset=3).run()                       # unaligned rows
    assert binding.last_path() == binding.PATH_STREAMING
    binding.set_path(binding.PATH_STREAMING)                  # and an explicit choice is honoured
    DeviceBatch(w).run()
    assert binding.last_path() == binding.PATH_STREAMING


def test_data_errors_and_next_lookahead():
    """Per-sequence data errors (bad token, bad temperature, negative or overrunning lookahead) give
    the oracle's status bits, -1 tokens and lookahead proposals; healthy neighbours are untouched."""
    w = W.make_config(2, B=6, V=4096, K=4)
    tok = w.draft_tokens.copy()
    tok[w.off_d[4] + 1] = 4096
    T = np.full(6, 0.8, np.float32)
    T[2] = 0.0
    c = Case(w.target_logits, w.draft_logits, tok, w.k_per_row, T, w.uniforms, dtype=w.dtype)
    got = DeviceBatch(c).run()
    assert binding.last_path() == binding.PATH_CLUSTER
    assert got[2].tolist() == [0, 0, 2, 0, 4, 0]
    assert_parity(c, got, max_excused_frac=0.2)
    for bad_b, new_k in ((5, 6), (1, -1)):                    # overruns the packed buffers; negative
        k = w.k_per_row.copy()
        k[bad_b] = new_k
        dev = DeviceBatch(w)
        dev.k = torch.from_numpy(k).cuda()
        nk = torch.full((6,), -9, dtype=torch.int32, device="cuda")
        binding.spec_verify(dev.target, dev.draft, dev.tokens, dev.k, dev.temperature, dev.uniforms,
                            accepted_len=dev.accepted, emitted_tokens=dev.emitted, row_status=dev.status,
                            next_k=nk, k_min=1, k_max=8)
        torch.cuda.synchronize()
        assert binding.last_path() == binding.PATH_CLUSTER
        acc, em, st = dev.accepted.cpu().numpy(), dev.emitted.cpu().numpy(), dev.status.cpu().numpy()
        ora = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, k, w.temperature, w.uniforms)
        assert np.array_equal(st & 7, ora.row_status & 7) and st[bad_b] == 1 and acc[bad_b] == 0
        good = (ora.row_status & 7) == 0
        assert np.array_equal(acc[good], ora.accepted_len[good])
        assert not np.any(em == -7), "every output slot is written"
        assert np.array_equal(nk.cpu().numpy(), oracle.next_lookahead(k, acc, 1, 8))
