"""Degenerate cases of the method on the GPU, both kernel sets, against the fp64 oracle through the
C ABI: a residual that is exactly zero (the fallback to the target row and its status bit), a
drafted token without draft mass, masked (-inf) logits, rows without any mass, and a second
uniform of exactly 1 (no cumulative value above the threshold).  The oracle's side of each case is
pinned in tests/test_oracle_hand_cases.py and tests/test_oracle_properties.py."""
import numpy as np
import pytest

from gpu_utils import DeviceBatch, assert_parity, run_oracle
from helpers import Case, masked_case, neg_inf_of
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("kernel_path")]

ZERO_RESIDUAL = binding.ROW_ZERO_RESIDUAL


def _expect_path(kernel_path, ring_capable=True):
    if kernel_path == "cluster":
        return                  # taken where the batch fits a cluster per sequence, else the automatic choice
    want = binding.PATH_RING if (kernel_path == "ring" and ring_capable) else binding.PATH_STREAMING
    assert binding.last_path() == want


@pytest.mark.parametrize("cfg,B,V", [(5, 24, 5000), (2, 40, 32000), (1, 20, 4096), (5, 9, 1001)])
def test_zero_residual_falls_back_to_the_target_row(kernel_path, cfg, B, V):
    """Every third sequence gets a draft row equal to its target row at some position and an accept
    uniform of exactly 1.0 there (outside the [0,1) contract, the only way to reject at ratio 1):
    u*q < p is false, the residual max(0, p-q) is zero everywhere, and the token must come from
    the target row itself with SPECV_ROW_ZERO_RESIDUAL set -- as the oracle does."""
    w = W.make_config(cfg, B=B, V=V)
    tl, dl, uni = w.target_logits, w.draft_logits.copy(), w.uniforms.copy()
    hit = {}
    for b in range(0, w.B, 3):
        K = int(w.k_per_row[b])
        i = b % K                                     # the position that is forced to reject
        for j in range(i + 1):                         # identical models up to and including it
            dl[w.off_d[b] + j] = tl[w.off_t[b] + j]
            uni[w.off_t[b] + j] = 0.25
        uni[w.off_t[b] + i] = 1.0
        hit[b] = i
    c = Case(tl, dl, w.draft_tokens, w.k_per_row, w.temperature, uni, dtype=w.dtype)
    got = DeviceBatch(c).run()
    _expect_path(kernel_path, ring_capable=(V * (4 if w.dtype == "f32" else 2)) % 16 == 0)
    ora = run_oracle(c)
    acc, em, st = got[0], got[1], got[2]
    for b, i in hit.items():
        assert ora.accepted_len[b] == i and ora.row_status[b] == ZERO_RESIDUAL
        assert acc[b] == i and st[b] == ZERO_RESIDUAL, f"sequence {b}"
    others = [b for b in range(w.B) if b not in hit]
    assert np.all(st[others] == 0)
    assert_parity(c, got, ora, max_excused_frac=0.1)


@pytest.mark.parametrize("cfg,B,V", [(5, 30, 20000), (1, 24, 4096), (2, 12, 32000)])
def test_masked_logits(kernel_path, cfg, B, V):
    """Half of every sequence's vocabulary at -inf (random ids, or one contiguous half so that whole
    vectors, lanes and chunks hold nothing else): masked tokens have probability exactly 0, are
    never emitted, and everything else agrees with the oracle as usual."""
    w = W.make_config(cfg, B=B, V=V)
    m, kept = masked_case(w, seed=cfg)
    got = DeviceBatch(m).run()
    _expect_path(kernel_path)
    assert_parity(m, got, max_excused_frac=0.1)
    acc, em = got[0], got[1]
    for b in range(m.B):
        token = em[m.off_t[b] + acc[b]]
        assert token in kept[b], f"sequence {b} emitted a masked token"


def test_rows_without_any_mass(kernel_path):
    """Rows made of -inf only.  A drafted token scored by such a target row is rejected and the draw
    falls through both the residual and the target row to the last token id (zero-residual bit
    set); an empty bonus row gives the last token id; an empty draft row rejects and the token
    comes from the target row."""
    w = W.make_config(5, B=30, V=8000)
    tl, dl, uni = w.target_logits.copy(), w.draft_logits.copy(), w.uniforms.copy()
    ninf = neg_inf_of(tl)
    ks = w.k_per_row
    a, b, c = [int(x) for x in np.nonzero(ks >= 3)[0][:3]]
    for s in (a, b, c):                                # identical models: everything is accepted ...
        dl[w.off_d[s]:w.off_d[s] + ks[s]] = tl[w.off_t[s]:w.off_t[s] + ks[s]]
    tl[w.off_t[a] + 1] = ninf                          # ... until the empty target row of position 1
    tl[w.off_t[b] + ks[b]] = ninf                      # empty bonus row
    dl[w.off_d[c]] = ninf                              # empty draft row at position 0
    case = Case(tl, dl, w.draft_tokens, ks, w.temperature, uni, dtype=w.dtype)
    got = DeviceBatch(case).run()
    _expect_path(kernel_path)
    ora = run_oracle(case)
    acc, em, st = got[0], got[1], got[2]
    assert acc[a] == 1 and em[w.off_t[a] + 1] == w.V - 1 and st[a] == ZERO_RESIDUAL
    assert acc[b] == ks[b] and em[w.off_t[b] + ks[b]] == w.V - 1 and st[b] == 0
    assert acc[c] == 0 and st[c] == ZERO_RESIDUAL
    for s in (a, b, c):
        assert acc[s] == ora.accepted_len[s] and st[s] == ora.row_status[s]
    assert_parity(case, got, ora, max_excused_frac=0.1)


@pytest.mark.parametrize("cfg,B,V", [(5, 24, 20000), (1, 12, 4096)])
def test_second_uniform_of_exactly_one(kernel_path, cfg, B, V):
    """u' = 1 for every sequence: no cumulative value lies strictly above the threshold, the draw is
    decided by the 'largest token id with mass' convention (hand cases H10a/b pin it exactly at
    V = 4).  At this size which id still has mass after rounding is not unique, so the check is:
    no fault, a valid token that has mass, lengths as the oracle's."""
    w = W.make_config(cfg, B=B, V=V)
    m, kept = masked_case(w, seed=7)                    # masks make 'last id with mass' != V - 1
    uni = m.uniforms.copy()
    uni[m.off_t + m.k_per_row] = 1.0
    m.uniforms = uni
    got = DeviceBatch(m).run()
    ora = run_oracle(m)
    assert np.all(ora.cdf_margin < 1e-9)                # the oracle itself calls every draw marginal
    assert_parity(m, got, ora, max_excused_frac=1.0)
    acc, em = got[0], got[1]
    for b in range(m.B):
        assert em[m.off_t[b] + acc[b]] in kept[b]
        if acc[b] == m.k_per_row[b]:                    # bonus draw: the last kept id has mass under p
            assert em[m.off_t[b] + acc[b]] >= kept[b][-1] - 512      # within the last segment that has mass


@pytest.mark.parametrize("cfg", [1, 2])      # fp32 and bf16 logits
def test_largest_vocabulary(kernel_path, cfg):
    """The largest vocabulary the library takes (2^22 entries: the segment table of the sampler is
    then at its shared-memory limit), two sequences: parity as usual; one entry more is refused."""
    V = 1 << 22
    w = W.make_config(cfg, B=2, V=V, K=2)
    got = DeviceBatch(w).run()
    assert_parity(w, got, max_excused_frac=0.5)
    assert binding.workspace_bytes(2, 4, V) > 0
    assert binding.workspace_bytes(2, 4, V + 1) == 0


def test_largest_vocabulary_tree():
    """Tree walk at 2^22 entries: fp32 logits (one CTA per sequence: two segment tables would not
    fit) and bf16 logits (pairs of CTAs)."""
    import test_gpu_tree as T
    for dtype in ("f32", "bf16"):
        w = W.make_tree_config(B=2, V=1 << 22, dtype=dtype, seed=31, depth=2, max_level_width=3)
        T.assert_tree_parity(w, T.run_gpu(w), max_excused_frac=0.5)


@pytest.mark.parametrize("B", [4095, 4096, 6000])
def test_batch_sizes_around_the_ring_kernels_limit(kernel_path, B):
    """The ring kernels keep one offset per sequence in shared memory and take up to 4095 sequences; a
    larger batch goes to the streaming kernels whatever the call asks for."""
    w = W.make_config(5, B=B, V=1024)
    got = DeviceBatch(w).run()
    _expect_path(kernel_path, ring_capable=B <= 4095)
    assert_parity(w, got, max_excused_frac=0.02)
