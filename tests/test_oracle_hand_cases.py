"""The oracle against values worked by hand (tests/golden/hand_cases.txt).

The paper's section "Speculative Sampling Results" gives the steps in prose and no
numbers; the fixture's numbers were derived by hand in exact fractions from the rule
the paper cites.  A dropped term, a swapped p/q, a wrong inequality direction or a
misplaced uniform changes at least one expected value below.
"""
import numpy as np
import pytest

import oracle
from helpers import hand_case_inputs, read_hand_cases

CASES = read_hand_cases()


def test_fixture_is_complete():
    assert len(CASES) >= 16
    assert {c["name"].split("_")[0].rstrip("ab") for c in CASES} >= {"H1", "H2", "H3", "H4", "H5", "H6", "H7", "H8",
                                                                       "H9", "H10"}


@pytest.mark.parametrize("case", CASES, ids=[c["name"] for c in CASES])
def test_hand_case(case):
    tl, dl, tok, k, T, uni = hand_case_inputs(case)
    res = oracle.spec_verify(tl, dl, tok, k, T, uni)
    assert res.row_status[0] == 0
    if case["zero_margin"]:
        # the draw sits on a CDF step: either neighbour is a legitimate floating-point
        # answer, and the oracle must say so through its margin
        assert res.cdf_margin[0] < 1e-6
        assert res.accepted_len[0] == case["expect_len"]
        return
    assert res.accepted_len[0] == case["expect_len"]
    assert res.emitted_tokens.tolist() == case["expect_emitted"]
    if case["no_crossing"]:
        # u' = 1: the threshold is the whole mass, so the draw is decided by the "largest id with
        # mass" convention (or by a last cumulative value that rounding put above the total)
        assert res.cdf_margin[0] < 1e-12
    elif case["u"][-1] > 0:   # u' = 0 touches the (empty) step below the first massive token
        assert res.cdf_margin[0] > 5e-4
    if "expect_ptok" in case:
        np.testing.assert_allclose(res.p_tok, case["expect_ptok"], rtol=1e-6)
        np.testing.assert_allclose(res.q_tok, case["expect_qtok"], rtol=1e-6)
        rho = (case["expect_rho"] if "expect_rho" in case
               else np.array(case["expect_ptok"]) / np.array(case["expect_qtok"]))
        np.testing.assert_allclose(res.rho, rho, rtol=1e-6)


def test_hand_cases_batched_ragged():
    """All hand cases with V=4 packed into ONE ragged batch give the same answers:
    pins the offset arithmetic (off_d, off_t) and the per-row temperature."""
    from helpers import pack, probs_to_logits
    cases = [c for c in CASES if not c["zero_margin"]]
    seqs = []
    for c in cases:
        K = len(c["tokens"])
        seqs.append({"target": probs_to_logits(c["target"]),
                     "draft": probs_to_logits(c["draft"]) if K else np.zeros((0, 4), np.float32),
                     "tokens": c["tokens"], "u": c["u"][:K], "u2": c["u"][K]})
    tl, dl, tok, k, uni, off_d, off_t = pack(seqs, 4)
    T = np.array([c["T"] for c in cases], np.float32)
    for threads in (1, 3):
        res = oracle.spec_verify(tl, dl, tok, k, T, uni, threads=threads)
        for b, c in enumerate(cases):
            K = int(k[b])
            assert res.accepted_len[b] == c["expect_len"], c["name"]
            assert res.emitted_tokens[off_t[b]:off_t[b] + K + 1].tolist() == c["expect_emitted"], c["name"]
