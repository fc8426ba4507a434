"""The oracle against invariants, special cases that reduce to library routines, and
a second, differently written formulation on thousands of tiny random inputs.

The steps being pinned are those of the paper's section "Speculative Sampling
Results": tokens are kept up to the first rejection and none after it; the rejected
token is resampled from a combination of both distributions; if all are accepted one
more token comes from the target distribution.
"""
import numpy as np
import pytest
from scipy.special import logsumexp

import oracle
from helpers import Case, bf16_bits_to_f64, f32_to_bf16_bits, logits_as_f64, masked_case, neg_inf_of, pack
from paper_2411_00853_b200 import workloads as W


def run(w, **kw):
    return oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.k_per_row,
                              w.temperature, w.uniforms, **kw)


# ---------------------------------------------------------------- second formulation
def second_formulation(tl, dl, tokens, u, u2, T):
    """One sequence, written differently from the C oracle: log-softmax through
    scipy's logsumexp, ratio through a difference of logs, inverse CDF through
    numpy's cumsum + searchsorted(side='right')."""
    K = len(tokens)
    lp = tl / T - logsumexp(tl / T, axis=1, keepdims=True)
    lq = dl / T - logsumexp(dl / T, axis=1, keepdims=True) if K else np.zeros((0, tl.shape[1]))
    for i in range(K):
        x = tokens[i]
        if not (np.log(u[i]) < lp[i, x] - lq[i, x] if u[i] > 0 else True):
            r = np.clip(np.exp(lp[i]) - np.exp(lq[i]), 0.0, None)
            c = np.cumsum(r)
            if c[-1] == 0.0:     # residual lost to rounding: the stated fallback is the target row
                c = np.cumsum(np.exp(lp[i]))
            return i, int(np.searchsorted(c, u2 * c[-1], side="right"))
    c = np.cumsum(np.exp(lp[K]))
    return K, int(np.searchsorted(c, u2 * c[-1], side="right"))


@pytest.mark.parametrize("V", [1, 2, 3, 7, 8, 9, 31, 33, 257])
@pytest.mark.parametrize("K", [0, 1, 2, 16])
def test_against_second_formulation(V, K):
    rng = np.random.default_rng(1000 * V + K)
    n_seq = 400
    seqs = []
    for _ in range(n_seq):
        T = 1.0
        tl = rng.normal(0, 3, (K + 1, V)).astype(np.float32)
        dl = (tl[:K] + rng.normal(0, 1.5, (K, V))).astype(np.float32)
        tokens = rng.integers(0, V, K)
        seqs.append({"target": tl, "draft": dl, "tokens": tokens,
                     "u": rng.random(K).astype(np.float32), "u2": np.float32(rng.random())})
    tl, dl, tok, k, uni, off_d, off_t = pack(seqs, V)
    T = rng.uniform(0.3, 1.5, n_seq).astype(np.float32)
    res = oracle.spec_verify(tl, dl, tok, k, T, uni)
    checked = 0
    for b, s in enumerate(seqs):
        thin = (np.nanmin(res.accept_margin[off_d[b]:off_d[b] + K], initial=1.0) < 1e-9
                or res.cdf_margin[b] < 1e-9)
        if thin:
            continue
        n, token = second_formulation(s["target"].astype(np.float64), s["draft"].astype(np.float64),
                                      s["tokens"], s["u"].astype(np.float64), float(s["u2"]),
                                      float(T[b]))
        assert res.accepted_len[b] == n
        assert res.emitted_tokens[off_t[b] + n] == token
        checked += 1
    assert checked > 0.95 * n_seq


def test_token_probabilities_match_library_softmax():
    w = W.make_config(2)
    res = run(w)
    for b in range(w.B):
        T = float(w.temperature[0])
        for i in range(int(w.k_per_row[b])):
            lt = logits_as_f64(w.target_logits[w.off_t[b] + i]) / T
            ld = logits_as_f64(w.draft_logits[w.off_d[b] + i]) / T
            x = w.draft_tokens[w.off_d[b] + i]
            p = np.exp(lt[x] - logsumexp(lt))
            q = np.exp(ld[x] - logsumexp(ld))
            np.testing.assert_allclose(res.p_tok[w.off_d[b] + i], p, rtol=1e-11)
            np.testing.assert_allclose(res.q_tok[w.off_d[b] + i], q, rtol=1e-11)
            np.testing.assert_allclose(res.rho[w.off_d[b] + i], p / q, rtol=1e-11)
            np.testing.assert_allclose(res.accept_margin[w.off_d[b] + i],
                                       abs(w.uniforms[w.off_t[b] + i] - p / q), rtol=1e-9, atol=1e-15)


# ---------------------------------------------------------------- invariants
def small_workloads():
    yield W.make_config(1)
    yield W.make_config(2)
    yield W.make_config(3, B=6, V=4096)
    yield W.make_config(4, B=12, V=3000)
    yield W.make_config(5, B=24, V=2051)


@pytest.mark.parametrize("w", list(small_workloads()), ids=lambda w: w.name)
def test_invariants(w):
    res = run(w, threads=4)
    assert np.all(res.row_status == 0)
    for b in range(w.B):
        K, n = int(w.k_per_row[b]), int(res.accepted_len[b])
        assert 0 <= n <= K                                             # accepted_len <= K_b
        em = res.emitted_tokens[w.off_t[b]:w.off_t[b] + K + 1]
        assert np.array_equal(em[:n], w.draft_tokens[w.off_d[b]:w.off_d[b] + n])   # prefix of the drafts
        assert 0 <= em[n] < w.V
        assert np.all(em[n + 1:] == -1)
        T = float(w.temperature[b] if w.temperature.shape[0] > 1 else w.temperature[0])
        # every accepted position really passed the test, position n really failed it
        u = w.uniforms[w.off_t[b]:w.off_t[b] + K].astype(np.float64)
        rho = res.rho[w.off_d[b]:w.off_d[b] + K]
        assert np.all(u[:n] < rho[:n])
        if n < K:
            assert u[n] >= rho[n]
            p, q, r = oracle.position_distributions(w.target_logits[w.off_t[b] + n],
                                                    w.draft_logits[w.off_d[b] + n], T)
            assert abs(p.sum() - 1) < 1e-12 and abs(q.sum() - 1) < 1e-12
            # sum max(0,p-q) = sum max(0,q-p) = 1 - sum min(p,q)
            assert abs(r.sum() - np.clip(q - p, 0, None).sum()) < 1e-12
            assert abs(r.sum() - (1 - np.minimum(p, q).sum())) < 1e-12
            y = em[n]
            assert p[y] > q[y] and y != w.draft_tokens[w.off_d[b] + n]   # resampled token has excess target mass


def test_later_uniforms_do_not_matter_and_length_is_monotone():
    w = W.make_config(5, B=12, V=777)
    base = run(w)
    rng = np.random.default_rng(7)
    uni = w.uniforms.copy()
    for b in range(w.B):
        K, n = int(w.k_per_row[b]), int(base.accepted_len[b])
        # scramble the accept uniforms after the first rejection
        uni[w.off_t[b] + n + 1:w.off_t[b] + K] = rng.random(max(0, K - n - 1)).astype(np.float32)
    again = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.k_per_row,
                               w.temperature, uni)
    assert np.array_equal(again.accepted_len, base.accepted_len)
    assert np.array_equal(again.emitted_tokens, base.emitted_tokens)
    # lowering every accept uniform can only lengthen, raising can only shorten
    lower, higher = w.uniforms.copy(), w.uniforms.copy()
    for b in range(w.B):
        K = int(w.k_per_row[b])
        lower[w.off_t[b]:w.off_t[b] + K] *= 0.5
        higher[w.off_t[b]:w.off_t[b] + K] = 0.5 + 0.5 * higher[w.off_t[b]:w.off_t[b] + K]
    lo = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.k_per_row, w.temperature, lower)
    hi = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.k_per_row, w.temperature, higher)
    assert np.all(lo.accepted_len >= base.accepted_len)
    assert np.all(hi.accepted_len <= base.accepted_len)


# ---------------------------------------------------------------- special cases
def numpy_sampler(logits_f64, T, u):
    z = logits_f64 / T
    p = np.exp(z - z.max())
    p /= p.sum()
    return int(np.searchsorted(np.cumsum(p), u, side="right"))


def test_identical_models_accept_everything_then_plain_sampling():
    """draft == target: every ratio is exactly 1, all K accepted, and the bonus token is
    an ordinary inverse-CDF softmax sample of the last target row."""
    w = W.make_config(2)
    dl = np.concatenate([w.target_logits[w.off_t[b]:w.off_t[b] + int(w.k_per_row[b])] for b in range(w.B)])
    res = oracle.spec_verify(w.target_logits, dl, w.draft_tokens, w.k_per_row, w.temperature, w.uniforms)
    assert np.all(res.rho == 1.0)
    assert np.array_equal(res.accepted_len, w.k_per_row)
    for b in range(w.B):
        K = int(w.k_per_row[b])
        u2 = float(w.uniforms[w.off_t[b] + K])
        if res.cdf_margin[b] < 1e-12:
            continue
        expect = numpy_sampler(bf16_bits_to_f64(w.target_logits[w.off_t[b] + K]), float(w.temperature[0]), u2)
        assert res.emitted_tokens[w.off_t[b] + K] == expect


def test_u_equal_to_ratio_rejects():
    """Strict inequality: with identical rows the ratio is exactly 1, and a uniform of
    exactly 1.0 (outside the [0,1) contract, used only to hit equality) must reject."""
    rng = np.random.default_rng(3)
    row = rng.normal(0, 2, (1, 16)).astype(np.float32)
    tl = np.concatenate([row, row])
    res = oracle.spec_verify(tl, row, np.array([5], np.int32), np.array([1], np.int32),
                             np.array([1.0], np.float32), np.array([1.0, 0.3], np.float32))
    assert res.accepted_len[0] == 0 and res.rho[0] == 1.0
    assert res.row_status[0] == oracle.ROW_ZERO_RESIDUAL   # p == q: nothing left to resample from
    assert res.emitted_tokens[0] == numpy_sampler(row[0].astype(np.float64), 1.0, 0.3)


def test_disjoint_supports_always_reject_and_resample_from_target():
    V, rng = 64, np.random.default_rng(11)
    seqs = []
    for _ in range(50):
        tl = rng.normal(0, 2, (2, V)).astype(np.float32)
        dl = rng.normal(0, 2, (1, V)).astype(np.float32)
        tl[:, V // 2:] = -1e30          # target lives on the first half
        dl[:, :V // 2] = -1e30          # draft on the second half
        seqs.append({"target": tl, "draft": dl, "tokens": [int(rng.integers(V // 2, V))],
                     "u": [np.float32(rng.random())], "u2": np.float32(rng.random())})
    tl, dl, tok, k, uni, off_d, off_t = pack(seqs, V)
    res = oracle.spec_verify(tl, dl, tok, k, np.array([0.9], np.float32), uni)
    assert np.all(res.accepted_len == 0) and np.all(res.rho == 0)
    for b, s in enumerate(seqs):
        if res.cdf_margin[b] < 1e-12:
            continue
        assert res.emitted_tokens[off_t[b]] == numpy_sampler(s["target"][0].astype(np.float64), 0.9, float(s["u2"]))


def test_no_draft_tokens_is_plain_sampling():
    V, rng = 100, np.random.default_rng(5)
    seqs = [{"target": rng.normal(0, 3, (1, V)).astype(np.float32), "draft": None, "tokens": [],
             "u": [], "u2": np.float32(rng.random())} for _ in range(64)]
    tl, dl, tok, k, uni, off_d, off_t = pack(seqs, V)
    res = oracle.spec_verify(tl, dl, tok, k, np.array([0.6], np.float32), uni)
    assert np.all(res.accepted_len == 0)
    for b, s in enumerate(seqs):
        assert res.emitted_tokens[off_t[b]] == numpy_sampler(s["target"][0].astype(np.float64), 0.6, float(s["u2"]))


def test_one_hot_target_always_emits_the_hot_token():
    V, rng = 50, np.random.default_rng(9)
    seqs = []
    for trial in range(40):
        hot = int(rng.integers(0, V))
        tl = np.full((2, V), -1e30, np.float32)
        tl[:, hot] = 0.0
        dl = rng.normal(0, 1, (1, V)).astype(np.float32)
        x = hot if trial % 2 else int(rng.integers(0, V))
        seqs.append({"target": tl, "draft": dl, "tokens": [x], "u": [np.float32(rng.random())],
                     "u2": np.float32(rng.random()), "hot": hot})
    tl, dl, tok, k, uni, off_d, off_t = pack(seqs, V)
    res = oracle.spec_verify(tl, dl, tok, k, np.array([1.0], np.float32), uni)
    for b, s in enumerate(seqs):
        assert res.emitted_tokens[off_t[b]] == s["hot"]            # accepted draft or resampled: the hot token
        if res.accepted_len[b] == 1:
            assert res.emitted_tokens[off_t[b] + 1] == s["hot"]    # bonus too


# ---------------------------------------------------------------- masked logits (-inf)
@pytest.mark.parametrize("cfg,V", [(1, 64), (5, 200), (2, 1024)])
def test_masked_logits_equal_the_compacted_vocabulary(cfg, V):
    """A logit of -inf is a token of probability 0 under either model, so masking half of the
    vocabulary must give exactly what the pass gives on the vocabulary with those ids removed:
    same accepted lengths, same probabilities of the drafted tokens, and emitted tokens that
    are the compacted run's tokens mapped back to the original ids."""
    w = W.make_config(cfg, B=18, V=V)
    m, kept = masked_case(w, seed=cfg)
    full = run(m)
    assert np.all(full.row_status == 0)
    # the compacted batch: every sequence keeps V // 2 ids, so the batch stays rectangular
    ctl = np.empty((m.target_logits.shape[0], V // 2), m.target_logits.dtype)
    cdl = np.empty((m.draft_logits.shape[0], V // 2), m.draft_logits.dtype)
    ctok = m.draft_tokens.copy()
    for b in range(m.B):
        K = int(m.k_per_row[b])
        ctl[m.off_t[b]:m.off_t[b] + K + 1] = m.target_logits[m.off_t[b]:m.off_t[b] + K + 1][:, kept[b]]
        cdl[m.off_d[b]:m.off_d[b] + K] = m.draft_logits[m.off_d[b]:m.off_d[b] + K][:, kept[b]]
        ctok[m.off_d[b]:m.off_d[b] + K] = np.searchsorted(kept[b], m.draft_tokens[m.off_d[b]:m.off_d[b] + K])
    small = oracle.spec_verify(ctl, cdl, ctok, m.k_per_row, m.temperature, m.uniforms)
    assert np.array_equal(full.accepted_len, small.accepted_len)
    np.testing.assert_allclose(full.p_tok, small.p_tok, rtol=1e-12)
    np.testing.assert_allclose(full.q_tok, small.q_tok, rtol=1e-12)
    checked = 0
    for b in range(m.B):
        if min(full.cdf_margin[b], small.cdf_margin[b]) < 1e-12:
            continue
        n = int(full.accepted_len[b])
        assert full.emitted_tokens[m.off_t[b] + n] == kept[b][small.emitted_tokens[m.off_t[b] + n]]
        assert not np.isneginf(logits_as_f64(m.target_logits[m.off_t[b] + n])[full.emitted_tokens[m.off_t[b] + n]])
        checked += 1
    assert checked >= m.B - 2


def test_rows_without_any_mass():
    """Degenerate rows made of -inf only (a mask that forbids everything) have no distribution.
    Stated behaviour: a drafted token scored by such a row is rejected; a draw from such a row
    yields the last token id; a residual that cannot be formed falls back to the target row and
    raises the zero-residual bit."""
    V, rng = 24, np.random.default_rng(21)
    ninf = np.float32(-np.inf)
    def seq(K):
        tl = rng.normal(0, 2, (K + 1, V)).astype(np.float32)
        return {"target": tl, "draft": tl[:K].copy(), "tokens": list(rng.integers(0, V, K)),
                "u": [np.float32(0.5)] * K, "u2": np.float32(0.4)}
    a, b, c, d = seq(2), seq(2), seq(2), seq(2)
    a["target"][1] = ninf                 # a: target row of position 1 empty -> rejected there, draw impossible
    b["target"][2] = ninf                 # b: identical models accept everything, the bonus row is empty
    c["draft"][0] = ninf                  # c: draft row of position 0 empty -> rejected, resampled from the target row
    tl, dl, tok, k, uni, off_d, off_t = pack([a, b, c, d], V)
    res = oracle.spec_verify(tl, dl, tok, k, np.array([1.0], np.float32), uni)
    assert res.accepted_len.tolist() == [1, 2, 0, 2]
    assert res.emitted_tokens[off_t[0] + 1] == V - 1 and res.row_status[0] == oracle.ROW_ZERO_RESIDUAL
    assert res.emitted_tokens[off_t[1] + 2] == V - 1 and res.row_status[1] == 0
    assert res.row_status[2] == oracle.ROW_ZERO_RESIDUAL
    assert res.emitted_tokens[off_t[2]] == numpy_sampler(c["target"][0].astype(np.float64), 1.0, 0.4)
    assert res.row_status[3] == 0


# ---------------------------------------------------------------- layout and data errors
def test_bf16_and_f32_storage_of_the_same_values_agree():
    w = W.make_config(5, B=8, V=1000)
    as_f32 = lambda a: (a.astype(np.uint32) << 16).view(np.float32)
    r16 = run(w)
    r32 = oracle.spec_verify(as_f32(w.target_logits), as_f32(w.draft_logits), w.draft_tokens,
                             w.k_per_row, w.temperature, w.uniforms)
    assert np.array_equal(r16.accepted_len, r32.accepted_len)
    assert np.array_equal(r16.emitted_tokens, r32.emitted_tokens)
    assert np.array_equal(r16.rho, r32.rho)


def test_padded_leading_dimension_and_threads_and_ranges():
    w = W.make_config(5, B=10, V=515)
    base = run(w)
    wide_t = np.full((w.target_logits.shape[0], 600), 0x7F80, np.uint16)   # +inf padding must never be read
    wide_d = np.full((w.draft_logits.shape[0], 640), 0x7F80, np.uint16)
    wide_t[:, :515], wide_d[:, :515] = w.target_logits, w.draft_logits
    padded = oracle.spec_verify(wide_t[:, :515], wide_d[:, :515], w.draft_tokens, w.k_per_row,
                                w.temperature, w.uniforms, threads=3)
    assert np.array_equal(padded.emitted_tokens, base.emitted_tokens)
    assert np.array_equal(padded.rho, base.rho)
    part = run(w, b_range=(3, 7))
    assert np.array_equal(part.accepted_len[3:7], base.accepted_len[3:7])
    assert np.all(part.accepted_len[:3] == -1) and np.all(part.accepted_len[7:] == -1)
    sub = run(w.take(3, 7))
    assert np.array_equal(sub.accepted_len, base.accepted_len[3:7])
    assert np.array_equal(sub.emitted_tokens, base.emitted_tokens[w.off_t[3]:w.off_t[7]])


def test_uniform_k_without_k_per_row():
    w = W.make_config(2)
    a = run(w)
    b = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, w.B, w.temperature,
                           w.uniforms, k_uniform=5)
    assert np.array_equal(a.emitted_tokens, b.emitted_tokens)


def test_data_errors_are_reported_per_row():
    w = W.make_config(5, B=6, V=300)
    tok = w.draft_tokens.copy()
    tok[w.off_d[1]] = 300                      # token out of range in sequence 1
    temp = np.full(6, 0.8, np.float32)
    temp[2], temp[4] = 0.0, np.inf             # bad temperatures in sequences 2 and 4
    res = oracle.spec_verify(w.target_logits, w.draft_logits, tok, w.k_per_row, temp, w.uniforms)
    good = run(w)
    assert res.row_status.tolist() == [0, oracle.ROW_BAD_TOKEN, oracle.ROW_BAD_TEMPERATURE, 0,
                                       oracle.ROW_BAD_TEMPERATURE, 0]
    for b in range(6):
        sl = slice(w.off_t[b], w.off_t[b] + int(w.k_per_row[b]) + 1)
        if res.row_status[b]:
            assert res.accepted_len[b] == 0 and np.all(res.emitted_tokens[sl] == -1)
        else:
            assert np.array_equal(res.emitted_tokens[sl], good.emitted_tokens[sl])
    # lookahead lengths that overrun the packed buffers
    k = w.k_per_row.copy()
    k[5] += 3
    res = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, k, w.temperature, w.uniforms)
    assert res.row_status[5] == oracle.ROW_BAD_K and np.all(res.row_status[:5] == 0)
    k = w.k_per_row.copy()
    k[0] = -2
    res = oracle.spec_verify(w.target_logits, w.draft_logits, w.draft_tokens, k, w.temperature, w.uniforms)
    assert res.row_status[0] == oracle.ROW_BAD_K and res.accepted_len[0] == 0


def test_generator_draws_tokens_from_the_draft_distribution():
    """The workload generator claims its tokens follow softmax(draft/T); check the claim
    with a chi-square-like bound on a tiny vocabulary (generator sanity, not the oracle)."""
    w = W.make_config(2, B=400, V=5, K=5)
    counts = np.zeros(5)
    expect = np.zeros(5)
    for d in range(w.n_draft_total):
        z = bf16_bits_to_f64(w.draft_logits[d]) / 0.7
        p = np.exp(z - logsumexp(z))
        expect += p
        counts[w.draft_tokens[d]] += 1
    assert np.all(np.abs(counts - expect) < 5 * np.sqrt(expect + 1))
    assert f32_to_bf16_bits(np.array([1.0, 1.00390625, 1.01171875], np.float32)).tolist() == [0x3F80, 0x3F80, 0x3F82]


def test_next_lookahead_rule_by_hand():
    """Hand-worked: all accepted -> +2, otherwise -1, clamped to [1, 8]; K = 0 counts as all accepted."""
    k = [4, 4, 1, 8, 7, 0, 3]
    n = [4, 2, 0, 8, 7, 0, 0]
    assert oracle.next_lookahead(k, n, 1, 8).tolist() == [6, 3, 1, 8, 8, 2, 2]
    assert oracle.next_lookahead(k, n, 0, 100).tolist() == [6, 3, 0, 10, 9, 2, 2]


def test_fp16_logits_decode_exactly():
    """Every finite binary16 bit pattern, through the oracle's decoder, against numpy's: a one-hot
    style probe (two-token vocabulary, the probed value against 0) returns softmax values that
    only the exact value reproduces; and fp16 storage equals fp32 storage of the same values."""
    bits = np.arange(0, 1 << 16, dtype=np.uint16)
    vals = bits.view(np.float16)
    finite = np.isfinite(vals) & (np.abs(vals.astype(np.float64)) < 600)   # keep exp() in range
    probe = vals[finite]
    tl = np.stack([probe, np.zeros_like(probe)], axis=1)                    # [n, 2] fp16
    for row16, row32 in zip(tl[::97], tl[::97].astype(np.float32)):
        p16, _, _ = oracle.position_distributions(row16, None, 1.0)
        p32, _, _ = oracle.position_distributions(row32, None, 1.0)
        assert np.array_equal(p16, p32)
    w = W.make_config(5, B=6, V=300, dtype="f16")
    a = run(w)
    b = oracle.spec_verify(w.target_logits.astype(np.float32), w.draft_logits.astype(np.float32), w.draft_tokens,
                           w.k_per_row, w.temperature, w.uniforms)
    assert np.array_equal(a.emitted_tokens, b.emitted_tokens) and np.array_equal(a.rho, b.rho)
