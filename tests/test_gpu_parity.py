"""CUDA library vs the fp64 oracle, through the C ABI, on the same seeded inputs.

Bar: accepted lengths and emitted tokens identical except where the oracle's own decision
margin (|u - ratio|, or the uniform's distance to a CDF step) is below 1e-5 -- those are
counted; per-position probabilities within 1e-5 relative.
"""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import DeviceBatch, assert_parity, run_oracle
from helpers import Case, hand_case_inputs, read_hand_cases
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("kernel_path")]


_Case = Case


@pytest.mark.parametrize("case", [c for c in read_hand_cases() if not c["zero_margin"]],
                         ids=lambda c: c["name"])
def test_hand_cases(kernel_path, case):
    w = _Case(*hand_case_inputs(case))
    acc, em, st, dp, dq = DeviceBatch(w).run()
    assert acc[0] == case["expect_len"] and em.tolist() == case["expect_emitted"] and st[0] == 0
    if kernel_path != "cluster":          # the cluster form takes the cases whose rows are whole 16-byte vectors
        assert binding.last_path() == (binding.PATH_RING if kernel_path == "ring" else binding.PATH_STREAMING)
    if "expect_ptok" in case:
        np.testing.assert_allclose(dp, case["expect_ptok"], rtol=1e-5)
        np.testing.assert_allclose(dq, case["expect_qtok"], rtol=1e-5)


@pytest.mark.parametrize("V", [1, 2, 3, 7, 8, 9, 31, 33, 257, 1000, 4099, 20000])
@pytest.mark.parametrize("cfg", [1, 2, 5])
def test_small_and_odd_vocabularies(cfg, V):
    """Spans no tile (V < one vector), several tiles and ragged tails, fp32 and bf16, fixed and
    ragged lookahead."""
    w = W.make_config(cfg, B=24, V=V)
    assert_parity(w, DeviceBatch(w).run(), max_excused_frac=0.1)


@pytest.mark.parametrize("ld_pad,elem_offset", [(0, 1), (3, 0), (5, 3), (8, 8), (1, 7)])
@pytest.mark.parametrize("cfg", [1, 5])
def test_unaligned_rows_and_padded_pitch(cfg, ld_pad, elem_offset):
    w = W.make_config(cfg, B=6, V=3001)
    ref = DeviceBatch(w).run()
    got = DeviceBatch(w, ld_pad=ld_pad, elem_offset=elem_offset).run()
    assert_parity(w, got)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])   # same answers as the aligned run


@pytest.mark.parametrize("K", [0, 1, 2, 16, 40])
def test_lookahead_extremes(K):
    w = W.make_config(2, B=5, V=2048, K=K)
    dev = DeviceBatch(w)
    assert_parity(w, dev.run())
    # the same batch through the k_per_row == NULL form
    got = dev.run(use_k_per_row=False, k_uniform=K)
    assert_parity(w, got)


def test_mixed_zero_and_long_lookahead():
    w = W.make_config(5, B=40, V=1500)
    k = w.k_per_row.copy()
    k[::5] = 0
    # rebuild a ragged batch with some K_b = 0 by dropping those sequences' draft rows
    keep_t, keep_d = [], []
    for b in range(w.B):
        keep_t += list(range(int(w.off_t[b]), int(w.off_t[b]) + int(k[b]) + 1))
        keep_d += list(range(int(w.off_d[b]), int(w.off_d[b]) + int(k[b])))
    c = _Case(w.target_logits[keep_t], w.draft_logits[keep_d], w.draft_tokens[keep_d], k,
              w.temperature, w.uniforms[keep_t], dtype="bf16")
    assert_parity(c, DeviceBatch(c).run())


@pytest.mark.parametrize("cfg", [1, 2])
def test_small_configs_full_size(cfg):
    w = W.make_config(cfg)
    assert_parity(w, DeviceBatch(w).run())


def test_identical_models_accept_everything():
    w = W.make_config(2, B=16)
    w.draft_logits = np.concatenate([w.target_logits[w.off_t[b]:w.off_t[b] + 5] for b in range(w.B)])
    acc, em, st, dp, dq = DeviceBatch(w).run()
    assert np.all(acc == 5)
    assert np.array_equal(dp, dq)
    assert_parity(w, (acc, em, st, dp, dq))


def test_data_errors_are_reported_not_faulted():
    w = W.make_config(5, B=8, V=900)
    tok = w.draft_tokens.copy()
    tok[w.off_d[1]] = 900
    tok[w.off_d[6] + int(w.k_per_row[6]) - 1] = -3
    temp = np.full(8, 0.8, np.float32)
    temp[2], temp[4] = -1.0, np.nan
    c = _Case(w.target_logits, w.draft_logits, tok, w.k_per_row, temp, w.uniforms, dtype="bf16")
    got = DeviceBatch(c).run()
    assert got[2].tolist() == [0, 4, 2, 0, 2, 0, 4, 0]
    assert_parity(c, got)
    # lookahead lengths that overrun the packed buffers, or are negative
    for bad_b, delta, in ((7, +2), (3, None)):
        k = w.k_per_row.copy()
        k[bad_b] = -1 if delta is None else k[bad_b] + delta
        dev = DeviceBatch(w)
        dev.k = torch.from_numpy(k).cuda()
        acc, em, st, _, _ = dev.run()
        ora = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, k, w.temperature, w.uniforms)
        assert np.array_equal(st & 7, ora.row_status & 7)
        assert st[bad_b] == 1 and acc[bad_b] == 0
        good = (ora.row_status & 7) == 0
        assert np.array_equal(acc[good], ora.accepted_len[good])


def test_runs_are_bit_identical():
    w = W.make_config(5, B=32, V=5000)
    dev = DeviceBatch(w)
    a = [x.copy() for x in dev.run()]
    b = dev.run()
    for x, y in zip(a, b):
        assert np.array_equal(x, y, equal_nan=True)


def test_host_entry_point_matches_device_entry_point():
    w = W.make_config(5, B=20, V=4000)
    ref = DeviceBatch(w).run()
    tl = torch.from_numpy(w.target_logits).view(torch.bfloat16).pin_memory()
    dl = torch.from_numpy(w.draft_logits).view(torch.bfloat16).pin_memory()
    arena = torch.empty(binding.host_arena_bytes(binding.BF16, w.B, w.n_draft_total, w.V), dtype=torch.uint8,
                        device="cuda")
    st = torch.empty(w.B, dtype=torch.int32).pin_memory()
    dp = torch.empty(w.n_draft_total, dtype=torch.float32).pin_memory()
    dq = torch.empty(w.n_draft_total, dtype=torch.float32).pin_memory()
    acc, em = binding.spec_verify_host(tl, dl, torch.from_numpy(w.draft_tokens), torch.from_numpy(w.k_per_row),
                                       torch.from_numpy(w.temperature), torch.from_numpy(w.uniforms), arena,
                                       row_status=st, diag_p_tok=dp, diag_q_tok=dq)
    assert np.array_equal(acc.numpy(), ref[0]) and np.array_equal(em.numpy(), ref[1])
    assert np.array_equal(st.numpy(), ref[2]) and np.array_equal(dp.numpy(), ref[3])


def test_argument_errors_come_back_as_status_codes():
    w = W.make_config(2, B=2, V=512)
    dev = DeviceBatch(w)
    lib = binding.load()

    def call(**over):
        import ctypes
        a = dict(tl=dev.target.data_ptr(), dl=dev.draft.data_ptr(), dtype=1, V=512, ldt=512, ldd=512,
                 tok=dev.tokens.data_ptr(), k=dev.k.data_ptr(), B=2, ku=0, D=10, T=dev.temperature.data_ptr(),
                 per=0, u=dev.uniforms.data_ptr(), acc=dev.accepted.data_ptr(), em=dev.emitted.data_ptr(),
                 ws=dev.workspace.data_ptr(), wsb=dev.workspace.numel())
        a.update(over)
        return lib.spec_verify(a["tl"], a["dl"], a["dtype"], a["V"], a["ldt"], a["ldd"], a["tok"], a["k"], a["B"],
                               a["ku"], a["D"], a["T"], a["per"], a["u"], a["acc"], a["em"], None, None, None,
                               a["ws"], a["wsb"], None)

    assert call() == 0
    assert call(tl=None) == 1 and call(u=None) == 1 and call(acc=None) == 1 and call(ws=None) == 1
    assert call(V=0) == 2 and call(B=0) == 2 and call(ldt=511) == 2 and call(D=-1) == 2
    assert call(k=None, ku=4) == 2            # B*k_uniform != n_draft_total
    assert call(dtype=3) == 3
    assert call(ws=dev.workspace.data_ptr() + 4) == 4 and call(tok=dev.tokens.data_ptr() + 2) == 4
    assert call(wsb=16) == 5

    def call_ex(flags, k_min=0, k_max=0, next_k=None):
        return lib.spec_verify_ex(dev.target.data_ptr(), dev.draft.data_ptr(), 1, 512, 512, 512,
                                  dev.tokens.data_ptr(), dev.k.data_ptr(), 2, 0, 10, dev.temperature.data_ptr(), 0,
                                  dev.uniforms.data_ptr(), dev.accepted.data_ptr(), dev.emitted.data_ptr(), None,
                                  None, None, dev.workspace.data_ptr(), dev.workspace.numel(), None, flags, k_min,
                                  k_max, next_k)

    assert call_ex(0) == 0 and call_ex(binding.FLAG_RING | binding.FLAG_EARLY_EXIT) == 0
    assert call_ex(binding.FLAG_RING | binding.FLAG_STREAMING) == 9 and call_ex(16) == 9 and call_ex(1 << 31) == 9
    assert call_ex(binding.FLAG_CLUSTER) == 0 and call_ex(binding.FLAG_CLUSTER | binding.FLAG_RING) == 9
    nk = torch.zeros(2, dtype=torch.int32, device="cuda")
    assert call_ex(0, 1, 8, nk.data_ptr()) == 0
    assert call_ex(0, -1, 8, nk.data_ptr()) == 2 and call_ex(0, 5, 4, nk.data_ptr()) == 2
    assert call_ex(0, 5, 4, None) == 0                    # the bounds only matter with next_k
    assert call_ex(0, 1, 8, nk.data_ptr() + 2) == 4
    torch.cuda.synchronize()


def test_kernel_set_selection(kernel_path):
    """The ring kernels are really the ones that run where the shape allows them (no silent
    fall-back), and shapes they cannot take go to the streaming kernels."""
    w = W.make_config(5, B=12, V=32000)
    DeviceBatch(w).run()
    assert binding.last_path() == {"ring": binding.PATH_RING, "streaming": binding.PATH_STREAMING,
                                   "cluster": binding.PATH_RING}[kernel_path]     # 100 draft rows: too many for the cluster form
    for V in (4099, 31):                       # rows that are not whole 16-byte vectors
        DeviceBatch(W.make_config(5, B=4, V=V)).run()
        assert binding.last_path() == binding.PATH_STREAMING
    DeviceBatch(w, elem_offset=3).run()        # unaligned rows
    assert binding.last_path() == binding.PATH_STREAMING
    binding.set_path(binding.PATH_AUTO)
    DeviceBatch(W.make_config(1)).run()        # one sequence whose rows fit a cluster's shared memory
    assert binding.last_path() == binding.PATH_CLUSTER
    DeviceBatch(W.make_config(1, V=200000)).run()        # 9 rows of 800 KB do not: 5 work items, streaming kernels
    assert binding.last_path() == binding.PATH_STREAMING
    DeviceBatch(W.make_config(5, B=64, V=32000)).run()
    assert binding.last_path() == binding.PATH_RING


def test_next_lookahead_matches_oracle(kernel_path):
    w = W.make_config(5, B=200, V=2048)
    dev = DeviceBatch(w)
    acc, *_ = dev.run()
    nxt = binding.next_lookahead(dev.k, dev.accepted, 1, 12).cpu().numpy()
    assert np.array_equal(nxt, oracle.next_lookahead(w.k_per_row, acc, 1, 12))
    uni = binding.next_lookahead(None, dev.accepted, 0, 9, k_uniform=3).cpu().numpy()
    assert np.array_equal(uni, oracle.next_lookahead(np.full(200, 3), acc, 0, 9))
    with pytest.raises(binding.SpecVerifyError):
        binding.next_lookahead(dev.k, dev.accepted, 5, 2)


@pytest.mark.parametrize("V", [5, 257, 4099, 20000, 32000])
@pytest.mark.parametrize("cfg", [2, 5])
def test_fp16_logits(kernel_path, cfg, V):
    w = W.make_config(cfg, B=24, V=V, dtype="f16")
    assert_parity(w, DeviceBatch(w).run(), max_excused_frac=0.1)
    assert DeviceBatch(w, ld_pad=3, elem_offset=1).run()[0].shape == (24,)


@pytest.mark.parametrize("cfg,B,V", [(2, 8, 32000), (5, 96, 32000)])
def test_a_pass_captured_in_a_cuda_graph_replays_to_the_same_outputs(kernel_path, cfg, B, V):
    """After one ordinary call (the library sets kernel attributes lazily, per device and dtype)
    a call only enqueues kernels on its stream, so it can be captured and replayed."""
    w = W.make_config(cfg, B=B, V=V)
    dev = DeviceBatch(w)
    ref = [x.copy() for x in dev.run()]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            binding.spec_verify(dev.target, dev.draft, dev.tokens, dev.k, dev.temperature, dev.uniforms,
                                accepted_len=dev.accepted, emitted_tokens=dev.emitted, row_status=dev.status,
                                diag_p_tok=dev.diag_p, diag_q_tok=dev.diag_q, workspace=dev.workspace,
                                stream=side.cuda_stream)
    torch.cuda.synchronize()
    for _ in range(3):
        dev.accepted.fill_(-7)
        dev.emitted.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(dev.accepted.cpu().numpy(), ref[0]) and np.array_equal(dev.emitted.cpu().numpy(), ref[1])
        assert np.array_equal(dev.status.cpu().numpy(), ref[2])
