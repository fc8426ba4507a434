"""spec_verify_from_hidden: the LM-head products on the tensor cores (tcgen05) with the row
statistics in their epilogue, then the resolve kernel.  Hidden states and weights are built so that
every product and sum is exactly representable: the oracle's fp64 product and any correct fp32
accumulation give the same bf16 bytes, so the logits are compared for EQUALITY and the verify
results against the oracle run on the oracle's own logits -- nothing the GPU produced goes into it."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import PROB_RTOL
from helpers import Case, classify_rows
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a)).view(torch.bfloat16).cuda()


def _oracle_side(w):
    tl = oracle.lm_head(w.target_hidden, w.target_weight, threads=16)
    dl = oracle.lm_head(w.draft_hidden, w.draft_weight, threads=16)
    tok = w.draw_tokens(dl)
    case = Case(tl, dl, tok, w.k_per_row, w.temperature, w.uniforms, dtype="bf16")
    ora = oracle.spec_verify(tl, dl, tok, w.k_per_row, w.temperature, w.uniforms, threads=16)
    return tl, dl, tok, case, ora


@pytest.mark.parametrize("B,V,H,Hd,K", [(6, 512, 64, 64, 2),          # one column tile pair, one k-block
                                         (20, 4096, 256, 128, None),   # several k-blocks, ragged lookahead
                                         (37, 20000, 320, 192, None),  # ragged last column tile, ragged last row tile, H not a multiple of 64
                                         (150, 2048, 128, 128, 3),     # many row tiles
                                         (32, 256, 64, 64, 3),         # exactly one 128 x 256 tile of target logits
                                         (43, 264, 192, 64, 2)])       # 129 target rows; 8 columns past a column tile
def test_logits_are_exact_and_the_pass_matches_the_oracle(B, V, H, Hd, K):
    w = W.make_hidden_config(B=B, V=V, H=H, Hd=Hd, K=K)
    tl, dl, tok, case, ora = _oracle_side(w)
    D = w.n_draft_total
    st = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    dp = torch.full((D,), float("nan"), device="cuda")
    dq = torch.full((D,), float("nan"), device="cuda")
    ws = torch.empty(binding.from_hidden_workspace_bytes(B, D, V), dtype=torch.uint8, device="cuda")
    acc, em, gtl, gdl = binding.spec_verify_from_hidden(
        _bf16(w.target_hidden), _bf16(w.target_weight), _bf16(w.draft_hidden), _bf16(w.draft_weight),
        torch.from_numpy(tok).cuda(), torch.from_numpy(w.k_per_row).cuda(), torch.from_numpy(w.temperature).cuda(),
        torch.from_numpy(w.uniforms).cuda(), row_status=st, diag_p_tok=dp, diag_q_tok=dq, workspace=ws)
    torch.cuda.synchronize()
    assert binding.from_hidden_status(ws, B, D, V) == 0
    # the products, byte for byte
    assert np.array_equal(gtl.view(torch.uint16).cpu().numpy().astype(np.uint16), tl)
    assert np.array_equal(gdl.view(torch.uint16).cpu().numpy().astype(np.uint16), dl)
    # the verify pass on them
    acc, em, st = acc.cpu().numpy(), em.cpu().numpy(), st.cpu().numpy()
    assert not st.any()
    np.testing.assert_allclose(dp.cpu().numpy(), ora.p_tok, rtol=PROB_RTOL, atol=1e-37)
    np.testing.assert_allclose(dq.cpu().numpy(), ora.q_tok, rtol=PROB_RTOL, atol=1e-37)
    identical, excused, failures = classify_rows(ora, w.k_per_row, acc, em, w.off_d, w.off_t)
    assert not failures and excused <= max(1, B // 10)


def test_random_hidden_states_agree_with_the_streaming_kernels_on_the_same_logits():
    """N(0,1) hidden states: the product is not exactly representable, so the logits are held to
    the oracle's within one bf16 unit in the last place (fp32 against fp64 accumulation), and the
    verify results to spec_verify run on the logits the call itself wrote."""
    w = W.make_hidden_config(B=24, V=8192, H=512, Hd=256, exact=False)
    D, B, V = w.n_draft_total, w.B, w.V
    tl = oracle.lm_head(w.target_hidden, w.target_weight, threads=16)
    dl = oracle.lm_head(w.draft_hidden, w.draft_weight, threads=16)
    tok = torch.from_numpy(w.draw_tokens(dl)).cuda()
    k, T, u = torch.from_numpy(w.k_per_row).cuda(), torch.from_numpy(w.temperature).cuda(), torch.from_numpy(w.uniforms).cuda()
    acc, em, gtl, gdl = binding.spec_verify_from_hidden(_bf16(w.target_hidden), _bf16(w.target_weight), _bf16(w.draft_hidden),
                                                        _bf16(w.draft_weight), tok, k, T, u)
    torch.cuda.synchronize()
    for got, want in ((gtl, tl), (gdl, dl)):
        g = got.float().cpu().numpy().astype(np.float64)
        x = (want.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        # one unit in the last place of the larger of the two, plus the absolute error of an fp32
        # accumulation over H terms (it decides the rounding of sums that cancel to nearly nothing)
        ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.maximum(np.abs(x), np.abs(g)), 1e-30))) - 7)
        assert np.all(np.abs(g - x) <= ulp * 1.0001 + 2e-5)
        assert (g == x).mean() > 0.97
    acc2, em2 = binding.spec_verify(gtl, gdl, tok, k, T, u, flags=binding.FLAG_STREAMING)
    torch.cuda.synchronize()
    same = (acc.cpu().numpy() == acc2.cpu().numpy())
    assert same.mean() >= 0.9         # the two statistics routes differ only in rounding; decisions agree but for thin margins


def test_shapes_the_products_cannot_take_are_refused():
    w = W.make_hidden_config(B=4, V=512, H=64, K=1)
    D, B, V = w.n_draft_total, w.B, w.V
    args = dict(draft_tokens=torch.zeros(D, dtype=torch.int32, device="cuda"), k_per_row=torch.from_numpy(w.k_per_row).cuda(),
                temperature=torch.from_numpy(w.temperature).cuda(), uniforms=torch.from_numpy(w.uniforms).cuda())
    th, tw, dh, dw = _bf16(w.target_hidden), _bf16(w.target_weight), _bf16(w.draft_hidden), _bf16(w.draft_weight)
    with pytest.raises(binding.SpecVerifyError) as e:       # hidden rows not on 16-byte boundaries
        wide = torch.zeros((D + B, 67), dtype=torch.bfloat16, device="cuda")
        binding.spec_verify_from_hidden(wide[:, :64], tw, dh, dw, args["draft_tokens"], args["k_per_row"],
                                        args["temperature"], args["uniforms"])
    assert e.value.status == 2
    with pytest.raises(binding.SpecVerifyError) as e:       # a vocabulary the ring kernels do not take
        binding.spec_verify_from_hidden(th, tw[:509], dh, dw[:509], args["draft_tokens"], args["k_per_row"],
                                        args["temperature"], args["uniforms"])
    assert e.value.status == 2
    torch.cuda.synchronize()
