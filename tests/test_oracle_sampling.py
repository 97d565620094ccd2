"""Pins of the oracle's sampling-based verification (Section 1: drafted tokens accepted so that the distribution of
the output equals the full model's; the T > 0 columns of Tables 3 and 4).

Each test ties a piece to something outside the oracle: the generator's published known-answer vectors, scipy's
softmax, numpy's cumulative sums, the closed form of the acceptance probability, the identity that makes the
method lossless in distribution (checked by a chi-square test over 10^5 rounds), and the greedy loop as the limit of
temperature zero.
"""
import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
import synth

SMALL = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)


# ------------------------------------------------------------------ the counter-based generator
def test_philox4x32_10_known_answers():
    # the three vectors published with the generator (Salmon et al., SC'11, reference implementation's known-answer
    # tests): all-zero input, all-one bits, and counter / key taken from the hexadecimal digits of pi
    def run(ctr, key):
        return [int(v) for v in oracle.philox4x32_10(ctr, key)]
    assert run([0, 0, 0, 0], [0, 0]) == [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]
    assert run([0xffffffff] * 4, [0xffffffff] * 2) == [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]
    assert run([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344], [0xa4093822, 0x299f31d0]) == \
        [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1]


def test_uniform_is_the_first_word_mapped_into_the_open_interval():
    seed, pos, kind = 0x0123456789abcdef, 77, oracle.DRAW_ACCEPT
    w = oracle.philox4x32_10([pos, kind, 0, 0], [seed & 0xffffffff, seed >> 32])
    assert oracle.uniform(seed, pos, kind) == (float(w[0]) + 0.5) / 2 ** 32
    # distinct streams per position and per kind, reproducible, inside (0, 1), and uniform (Kolmogorov-Smirnov)
    u = np.array([oracle.uniform(5, p, k) for p in range(4000) for k in range(3)])
    assert u.min() > 0 and u.max() < 1 and len(set(u.tolist())) == u.size
    assert scipy.stats.kstest(u, "uniform").pvalue > 1e-3
    assert oracle.uniform(5, 10, 1) == oracle.uniform(5, 10, 1) != oracle.uniform(6, 10, 1)


# ------------------------------------------------------------------ softmax at a temperature, inverse-CDF sampling
def test_softmax_with_temperature_equals_scipy():
    rng = np.random.default_rng(0)
    logits = rng.normal(0, 3, 1000).astype(np.float32)
    for T in (0.2, 0.6, 1.0, 5.0):
        ref = scipy.special.softmax(logits.astype(np.float64) / T)
        np.testing.assert_allclose(oracle.softmax_t(logits, T), ref, rtol=1e-12, atol=0)
    big = np.array([1000.0, 999.0, -1000.0], np.float32)            # no overflow: the maximum is subtracted
    np.testing.assert_allclose(oracle.softmax_t(big, 1.0), scipy.special.softmax(big.astype(np.float64)), rtol=1e-12)


def test_inverse_cdf_sampling_equals_numpy_searchsorted():
    rng = np.random.default_rng(1)
    w = rng.random(200)
    w[rng.integers(0, 200, 40)] = 0.0                                  # zero-weight entries are never chosen
    cdf = np.cumsum(w)
    for u in rng.random(500):
        got = oracle.sample_cdf(w, u)
        assert got == int(np.searchsorted(cdf, u * cdf[-1], side="right")) and w[got] > 0
    # unnormalised weights give the same draw; the ends of the interval stay inside the support
    assert oracle.sample_cdf(3 * w, 0.37) == oracle.sample_cdf(w, 0.37)
    assert w[oracle.sample_cdf(w, 1e-12)] > 0 and w[oracle.sample_cdf(w, 1 - 1e-12)] > 0
    assert oracle.sample_cdf(np.array([0.0, 0.0, 2.0, 0.0]), 0.999999) == 2


# ------------------------------------------------------------------ the acceptance rule
def test_identical_distributions_accept_every_draft():
    rng = np.random.default_rng(2)
    V, k = 11, 5
    p = rng.random((k + 1, V)); p /= p.sum(1, keepdims=True)
    for seed in range(50):
        drafts = [oracle.sample_cdf(p[j], oracle.uniform(seed, 100 + 1 + j, oracle.DRAW_DRAFT)) for j in range(k)]
        a, out = oracle.spec_accept(p, p[:k], drafts, seed, 100)
        assert a == k and out[:k].tolist() == drafts
        # the extra token is a TARGET draw from the last row
        assert out[k] == oracle.sample_cdf(p[k], oracle.uniform(seed, 100 + 1 + k, oracle.DRAW_TARGET))


def test_acceptance_threshold_and_residual_distribution():
    # one draft, V = 3: p = (0.5, 0.3, 0.2), q = (0.2, 0.7, 0.1). Draft token 1 is accepted iff its ACCEPT draw is below
    # p/q = 3/7; on rejection the replacement comes from max(0, p - q) / 0.4 = (0.75, 0, 0.25). Draft token 0 (p > q) is
    # always accepted.
    p = np.array([[0.5, 0.3, 0.2], [1 / 3, 1 / 3, 1 / 3]])
    q = np.array([[0.2, 0.7, 0.1]])
    n_acc = n_rej = 0
    for seed in range(400):
        r = oracle.uniform(seed, 8, oracle.DRAW_ACCEPT)
        a, out = oracle.spec_accept(p, q, [1], seed, 7)
        if r < 3 / 7:
            assert a == 1 and out[0] == 1
            n_acc += 1
        else:
            u = oracle.uniform(seed, 8, oracle.DRAW_TARGET)
            assert a == 0 and out.tolist() == [0 if u < 0.75 else 2]
            n_rej += 1
        a0, out0 = oracle.spec_accept(p, q, [0], seed, 7)
        assert a0 == 1 and out0[0] == 0
    assert n_acc > 100 and n_rej > 150


def test_emitted_tokens_follow_the_full_models_distribution_for_a_wrong_draft_model():
    # The identity behind the method: min(p, q)(x) + (1 - sum min(p, q)) * res(x) = p(x). Position-independent p and a
    # deliberately different q; over 10^5 rounds the first emitted token must be distributed as p (chi-square), and
    # so must the second one given that the first draft was accepted.
    rng = np.random.default_rng(3)
    V, k, N = 8, 3, 100_000
    p_row = rng.random(V) ** 2; p_row /= p_row.sum()
    q_row = rng.random(V) ** 2; q_row /= q_row.sum()
    p, q = np.tile(p_row, (k + 1, 1)), np.tile(q_row, (k, 1))
    first = np.zeros(V); second = np.zeros(V); accepted = 0
    for s in range(N):
        drafts = [oracle.sample_cdf(q_row, oracle.uniform(s, 1 + j, oracle.DRAW_DRAFT)) for j in range(k)]
        a, out = oracle.spec_accept(p, q, drafts, s, 0)
        first[out[0]] += 1
        if a >= 1:
            second[out[1]] += 1
        accepted += a
    assert scipy.stats.chisquare(first, p_row * N).pvalue > 1e-3
    assert scipy.stats.chisquare(second, p_row * second.sum()).pvalue > 1e-3
    # a draft is accepted with probability sum_x min(p, q): the expected accepted length is b + b^2 + b^3
    b = np.minimum(p_row, q_row).sum()
    assert accepted / N == pytest.approx(b + b ** 2 + b ** 3, abs=0.02)
    # plain sampling from q would NOT pass: the test has power against a missing correction
    assert scipy.stats.chisquare(np.bincount([oracle.sample_cdf(q_row, oracle.uniform(s, 1, 0)) for s in range(20000)],
                                             minlength=V), p_row * 20000).pvalue < 1e-6


# ------------------------------------------------------------------ the decoding loops with sampling
@pytest.fixture(scope="module")
def small():
    return synth.make_model(SMALL, seed=7, std=0.2)


def test_vanishing_temperature_gives_the_greedy_loop(small):
    o = oracle.Oracle(small, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=9)
    greedy, margins, _ = o.generate(prompt, 24, mode=oracle.MODE_AR)
    # T = 1e-4: the softmax puts all mass on the argmax wherever the top-2 gap is far above T
    cold_ar, _, _ = o.generate(prompt, 24, mode=oracle.MODE_AR, temperature=1e-4, seed=3)
    assert margins.min() > 30 * 1e-4 and cold_ar.tolist() == greedy.tolist()      # exp(-30) of the mass elsewhere at most
    o.set_skip_mask([0, 1], [1, 0])
    cold_sp, _, st = o.generate(prompt, 24, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4, temperature=1e-4, seed=3)
    assert cold_sp.tolist() == greedy.tolist()
    o.set_skip_mask([0, 1], [1, 0])
    _, _, st0 = o.generate(prompt, 24, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4)
    assert st["accepted"] == st0["accepted"] and st["drafted"] == st0["drafted"]   # the same rounds as greedy verification


def test_empty_mask_accepts_every_sampled_draft_and_reproduces_plain_sampling(small):
    # D = M: q = p, so every draft is accepted; the drafted token at a position is a DRAFT draw while plain sampling uses
    # the TARGET draw there, so the two sequences differ, but both are reproducible and differ between seeds
    o = oracle.Oracle(small, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=10)
    o.set_skip_mask([0, 0], [0, 0])
    a, _, st = o.generate(prompt, 30, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4, temperature=0.8, seed=11)
    assert st["accepted"] == st["drafted"] > 0
    o.set_skip_mask([0, 0], [0, 0])
    b, _, _ = o.generate(prompt, 30, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4, temperature=0.8, seed=11)
    assert a.tolist() == b.tolist()
    c, _, _ = o.generate(prompt, 30, mode=oracle.MODE_AR, temperature=0.8, seed=11)
    d, _, _ = o.generate(prompt, 30, mode=oracle.MODE_AR, temperature=0.8, seed=12)
    assert c.tolist() != d.tolist()


def test_sampled_generation_replays_through_the_single_step_calls(small):
    # the loop is the composition of its steps: draft steps (which keep q), one verify (which applies the rule)
    o = oracle.Oracle(small, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 5, seed=12)
    T, seed, k = 0.7, 21, 3
    o.set_skip_mask([1, 0], [0, 1])
    want, _, st = o.generate(prompt, 16, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=k, temperature=T, seed=seed)
    r = oracle.Oracle(small, max_seq=64)
    r.set_sampling(T, seed)
    got = [r.prefill(prompt)]
    r.set_skip_mask([1, 0], [0, 1])
    while len(got) < 16:
        kk = min(k, 16 - len(got) - 1)
        row = [got[-1]]
        for _ in range(kk):
            row.append(r.draft_step(row[-1]))
        a, out = r.verify(row)
        got += out.tolist()
    assert got[:16] == want.tolist()
    assert 0 < st["accepted"] < st["drafted"]                      # this mask gets some drafts rejected and some accepted


def test_first_emitted_token_of_the_model_follows_p_under_a_masked_draft(small):
    # end to end on the decoder: 4000 seeds, the token emitted at the first generated position after t_1 must follow
    # softmax(logits / T) of the FULL model although it is drafted by a sub-network
    o = oracle.Oracle(small, max_seq=32)
    prompt = synth.make_prompt(SMALL.vocab, 5, seed=13)
    T = 1.5
    greedy_first = o.prefill(prompt)
    o.reset()
    o.prefill(prompt)
    o.decode_step(greedy_first)
    p = oracle.softmax_t(o.last()["logits"][0], T)
    counts = np.zeros(SMALL.vocab)
    n = 4000
    for s in range(n):
        o.reset()
        o.set_sampling(0.0)
        t1 = o.prefill(prompt)                                       # greedy first token: the same context for every seed
        o.set_sampling(T, s)
        o.set_skip_mask([1, 1], [0, 1])
        d = o.draft_step(t1)
        a, out = o.verify([t1, d])
        counts[out[0]] += 1
    keep = p * n >= 5                                                # chi-square needs expected counts of at least ~5
    obs, exp = counts[keep], p[keep] * n
    if (~keep).any():
        obs, exp = np.append(obs, counts[~keep].sum()), np.append(exp, p[~keep].sum() * n)
    assert scipy.stats.chisquare(obs, exp).pvalue > 1e-3


def test_verify_with_sampling_needs_the_drafts_of_this_round(small):
    o = oracle.Oracle(small, max_seq=32)
    o.set_sampling(0.9, 1)
    t = o.prefill([1, 2, 3])
    with pytest.raises(oracle.OracleError) as e:
        o.verify([t, 4, 5])                                          # nothing was drafted: q is unknown
    assert e.value.code == oracle.ERR_STATE
    d = o.draft_step(t)
    with pytest.raises(oracle.OracleError) as e:
        o.verify([t, (d + 1) % SMALL.vocab])                         # not the token that was drafted
    assert e.value.code == oracle.ERR_STATE
    a, out = o.verify([t, d])
    assert 0 <= a <= 1 and len(out) == a + 1
