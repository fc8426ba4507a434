"""Per-call options of spec_verify_ex: the library keeps no mode between calls, so host threads
with different options do not interfere; the lookahead of the next round can be written by the
pass itself."""
import threading

import numpy as np
import pytest
import torch

import oracle
from gpu_utils import DeviceBatch, assert_parity, run_oracle
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run(dev: DeviceBatch, flags, stream, next_k=None, k_min=0, k_max=0):
    binding.spec_verify(dev.target, dev.draft, dev.tokens, dev.k, dev.temperature, dev.uniforms,
                        accepted_len=dev.accepted, emitted_tokens=dev.emitted, row_status=dev.status,
                        diag_p_tok=dev.diag_p, diag_q_tok=dev.diag_q, workspace=dev.workspace,
                        stream=stream.cuda_stream, flags=flags, next_k=next_k, k_min=k_min, k_max=k_max)


def test_two_host_threads_with_different_options_at_the_same_time():
    """Thread A runs the streaming kernels, thread B the ring kernels with early exit, each on its own
    batch, workspace and stream, many passes interleaved.  Each thread sees its own kernel set
    (spec_verify_last_path is per thread) and both results match the oracle."""
    wa, wb = W.make_config(5, B=70, V=20000), W.make_config(2, B=40, V=32000)
    da, db = DeviceBatch(wa), DeviceBatch(wb)
    torch.cuda.synchronize()
    seen, errors = {}, []
    start = threading.Barrier(2)

    def worker(name, dev, flags):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            start.wait()
            paths = set()
            for _ in range(40):
                _run(dev, flags, stream)
                paths.add(binding.last_path())
            stream.synchronize()
            seen[name] = paths
        except Exception as e:          # pragma: no cover - reported below
            errors.append((name, e))

    ta = threading.Thread(target=worker, args=("a", da, binding.FLAG_STREAMING))
    tb = threading.Thread(target=worker, args=("b", db, binding.FLAG_RING | binding.FLAG_EARLY_EXIT))
    ta.start(); tb.start(); ta.join(); tb.join()
    assert not errors, errors
    assert seen == {"a": {binding.PATH_STREAMING}, "b": {binding.PATH_RING}}
    torch.cuda.synchronize()
    for w, d in ((wa, da), (wb, db)):
        acc, em, st = d.accepted.cpu().numpy(), d.emitted.cpu().numpy(), d.status.cpu().numpy()
        ora = run_oracle(w)
        from helpers import classify_rows
        _, _, failures = classify_rows(ora, w.k_per_row, acc, em, w.off_d, w.off_t)
        assert not failures and not (st & ~15).any()
    # thread A's batch was fully evaluated, so its probabilities are all there
    assert_parity(wa, (da.accepted.cpu().numpy(), da.emitted.cpu().numpy(), da.status.cpu().numpy(),
                       da.diag_p.cpu().numpy(), da.diag_q.cpu().numpy()))


@pytest.mark.parametrize("flags", [binding.FLAG_STREAMING, binding.FLAG_RING,
                                   binding.FLAG_RING | binding.FLAG_EARLY_EXIT])
def test_next_lookahead_written_by_the_pass(flags):
    """next_k from inside the pass equals the oracle's rule on the pass's own accepted lengths, for
    valid sequences and for sequences with data errors, and costs no extra launch."""
    w = W.make_config(5, B=150, V=4096)
    tok = w.draft_tokens.copy()
    tok[w.off_d[4]] = 4096                               # bad token
    temp = np.full(w.B, 0.8, np.float32)
    temp[9] = -1.0                                       # bad temperature
    k = w.k_per_row.copy()
    k[w.B - 1] += 5                                      # lookahead overruns the buffers
    w.draft_tokens, w.temperature = tok, temp
    dev = DeviceBatch(w)
    dev.k = torch.from_numpy(k).cuda()
    stream = torch.cuda.current_stream()
    _run(dev, flags, stream)                             # lazy per-device set-up outside the count
    nk = torch.full((w.B,), -5, dtype=torch.int32, device="cuda")
    before = binding.launch_count()
    _run(dev, flags, stream, next_k=nk, k_min=1, k_max=12)
    launches_with = binding.launch_count() - before
    before = binding.launch_count()
    _run(dev, flags, stream)
    assert binding.launch_count() - before == launches_with
    torch.cuda.synchronize()
    acc, st = dev.accepted.cpu().numpy(), dev.status.cpu().numpy()
    assert st[4] == 4 and st[9] == 2 and st[w.B - 1] == 1
    assert np.array_equal(nk.cpu().numpy(), oracle.next_lookahead(k, acc, 1, 12))
    # and the same numbers as the stand-alone entry point
    assert np.array_equal(nk.cpu().numpy(), binding.next_lookahead(dev.k, dev.accepted, 1, 12).cpu().numpy())


def test_uniform_lookahead_without_k_per_row():
    w = W.make_config(2, B=64, V=2048, K=3)
    dev = DeviceBatch(w)
    nk = torch.full((w.B,), -5, dtype=torch.int32, device="cuda")
    for flags in (binding.FLAG_STREAMING, binding.FLAG_RING):
        binding.spec_verify(dev.target, dev.draft, dev.tokens, None, dev.temperature, dev.uniforms, k_uniform=3,
                            accepted_len=dev.accepted, emitted_tokens=dev.emitted, workspace=dev.workspace,
                            flags=flags, next_k=nk, k_min=0, k_max=4)
        torch.cuda.synchronize()
        acc = dev.accepted.cpu().numpy()
        assert np.array_equal(nk.cpu().numpy(), oracle.next_lookahead(np.full(w.B, 3), acc, 0, 4))


def test_greedy_and_tree_take_the_kernel_set_per_call():
    w = W.make_config(5, B=80, V=4096)
    dev = DeviceBatch(w)
    for flags, path in ((binding.FLAG_STREAMING, binding.PATH_STREAMING), (binding.FLAG_RING, binding.PATH_RING)):
        binding.spec_verify_greedy(dev.target, dev.tokens, dev.k, flags=flags)
        assert binding.last_path() == path
    # early exit is an option of spec_verify_ex alone (the wrapper masks the bit: raw C ABI here)
    lib = binding.load()
    ws = torch.empty(max(256, binding.greedy_workspace_bytes(w.B, w.n_draft_total)), dtype=torch.uint8, device="cuda")
    rc = lib.spec_verify_greedy(dev.target.data_ptr(), 1, w.V, w.V, dev.tokens.data_ptr(), dev.k.data_ptr(), w.B, 0,
                                w.n_draft_total, dev.accepted.data_ptr(), dev.emitted.data_ptr(), None, None,
                                ws.data_ptr(), ws.numel(), None, binding.FLAG_EARLY_EXIT)
    assert rc == 9 and "flag" in binding.strerror(9)
    torch.cuda.synchronize()
