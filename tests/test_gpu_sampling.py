"""GPU parity of sampling-based decoding and verification (Section 1; Tables 3 and 4 at T = 0.2 / 0.6) against the oracle.

Both sides evaluate softmax(logits / T), the acceptance test r q(x) < p(x) and the inverse-CDF search in double
precision with the same counter-based generator, so their choices can only differ through the logits (float32
accumulation on the GPU against double in the oracle, up to the logit tolerance). A choice is "decided" when the
oracle's uniform number is farther than MARGIN_U from the threshold that it is compared with (the two ends of the
chosen token's interval of the cumulative distribution; p/q for an acceptance test); every decided choice must be
identical on the GPU, and the tests count them.
"""
import numpy as np
import pytest

import oracle
import synth
from helpers import assert_logits_close

pytestmark = pytest.mark.gpu

MID = synth.DecoderShape(n_layers=3, d_model=512, n_heads=4, head_dim=128, d_ffn=1376, vocab=3001)
# The margin in u. The GPU's logits differ from the oracle's by float32 accumulation and by inherited one-ulp bf16
# flips of intermediate activations; the resulting shift of a cumulative probability stays below this on the models used.
MARGIN_U = 1e-3
# Weights with a larger spread than the default recipe: the logits then spread over several units, as a trained model's
# do, so that most draws fall on tokens whose probability interval is much wider than the margin (with the default
# recipe at vocabulary 1024 nearly every token's interval is narrower than 1e-3 at T = 0.6 and nothing would be decided).
SHARP_STD = 0.08


def _pair(shape, model, max_seq):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(shape, max_seq=max_seq, max_draft=8)
    dec.load_weights_host(model)
    return dec, oracle.Oracle(model, max_seq=max_seq)


def _draw_margin(probs, u):
    """(token, distance of u to the nearer end of the token's interval of the cumulative distribution)."""
    cdf = np.cumsum(probs)
    tok = oracle.sample_cdf(probs, u)
    lo = cdf[tok - 1] / cdf[-1] if tok > 0 else 0.0
    hi = cdf[tok] / cdf[-1]
    return tok, min(u - lo, hi - u)


@pytest.fixture(scope="module")
def sharp_tiny():
    return synth.make_model(synth.TINY, seed=0, std=SHARP_STD)


def _verify_margin(p, q, drafts, seed, pos0):
    """Smallest distance between a uniform number and the threshold it is compared with, over the choices of one round."""
    worst = 1.0
    for j, x in enumerate(drafts):
        r = oracle.uniform(seed, pos0 + 1 + j, oracle.DRAW_ACCEPT)
        ratio = p[j][x] / q[j][x]
        if ratio < 1.0:
            worst = min(worst, abs(r - ratio))
        if r * q[j][x] < p[j][x]:
            continue
        res = np.maximum(0.0, p[j] - q[j])
        return min(worst, _draw_margin(res, oracle.uniform(seed, pos0 + 1 + j, oracle.DRAW_TARGET))[1])
    k = len(drafts)
    return min(worst, _draw_margin(p[k], oracle.uniform(seed, pos0 + 1 + k, oracle.DRAW_TARGET))[1])


def _verify_decided(p_o, q_o, p_g, q_g, drafts, seed, pos0):
    """True when no choice of the oracle's verification of this round can come out differently on the GPU's
    distributions: every acceptance test has its uniform number outside the interval between the two sides' ratios
    p(x)/q(x) (and MARGIN_U away from the oracle's), and the final draw is farther from the ends of its token's interval
    than the L1 distance of the two sides' (normalised) distributions, which bounds the shift of every cumulative sum."""
    def draw_ok(w_o, w_g, u):
        w_o, w_g = w_o / w_o.sum(), w_g / w_g.sum()
        return _draw_margin(w_o, u)[1] > max(MARGIN_U, np.abs(w_o - w_g).sum())
    for j, x in enumerate(drafts):
        r = oracle.uniform(seed, pos0 + 1 + j, oracle.DRAW_ACCEPT)
        ratio_o, ratio_g = p_o[j][x] / q_o[j][x], p_g[j][x] / q_g[j][x]
        if min(ratio_o, ratio_g) < 1.0 and abs(r - min(1.0, ratio_o)) <= max(MARGIN_U, abs(ratio_o - ratio_g)):
            return False
        if r * q_o[j][x] < p_o[j][x]:
            continue
        return draw_ok(np.maximum(0.0, p_o[j] - q_o[j]), np.maximum(0.0, p_g[j] - q_g[j]), oracle.uniform(seed, pos0 + 1 + j, oracle.DRAW_TARGET))
    k = len(drafts)
    return draw_ok(p_o[k], p_g[k], oracle.uniform(seed, pos0 + 1 + k, oracle.DRAW_TARGET))


@pytest.mark.parametrize("which,T", [("tiny", 0.6), ("tiny", 0.2), ("mid", 0.3)])
def test_sampled_draft_and_verify_steps_match_oracle(which, T, sharp_tiny, tiny_prompt):
    """Two comparisons per choice. (1) The rule itself: the oracle's softmax / inverse-CDF / acceptance functions applied
    to the GPU's OWN logits must give exactly the GPU's choice (both sides work in double; only a uniform number within
    1e-9 of a threshold is left out). (2) End to end: the GPU's choice equals the oracle's wherever the oracle's uniform
    number is farther from its threshold than the two distributions differ (their L1 distance bounds the shift of
    every cumulative probability) and than MARGIN_U."""
    import paper_2410_01028_b200 as asd
    if which == "tiny":
        shape, model, prompt = synth.TINY, sharp_tiny, tiny_prompt
        mask = ([0, 1, 0, 0], [0, 0, 1, 0])
    else:
        shape, model = MID, synth.make_model(MID, seed=3, std=0.1)
        prompt = synth.make_prompt(MID.vocab, 70, seed=2)
        mask = ([0, 1, 0], [1, 0, 0])
    dec, orc = _pair(shape, model, max_seq=len(prompt) + 80)
    exact = decided_draws = decided_rounds = rounds = 0

    def check_draw(tok_gpu, lg_gpu, lg_orc, tok_orc, u):
        nonlocal exact, decided_draws
        p_g, p_o = oracle.softmax_t(lg_gpu, T), oracle.softmax_t(lg_orc, T)
        tok_rule, m_rule = _draw_margin(p_g, u)
        if m_rule > 1e-9:
            assert tok_gpu == tok_rule
            exact += 1
        tok, m_o = _draw_margin(p_o, u)
        assert tok == tok_orc
        if m_o > max(MARGIN_U, np.abs(p_g - p_o).sum()):
            assert tok_gpu == tok_orc
            decided_draws += 1
        return p_g, p_o

    for seed in (1, 2, 3, 4):
        dec.reset(); orc.reset()
        dec.set_debug(True)
        dec.set_sampling(T, seed); orc.set_sampling(T, seed)
        t_g, t_o = dec.prefill(prompt), orc.prefill(prompt)
        assert_logits_close(dec.get_last_logits()[-1:], orc.last()["logits"][-1:])
        check_draw(t_g, dec.get_last_logits()[-1], orc.last()["logits"][-1], t_o, oracle.uniform(seed, len(prompt), oracle.DRAW_TARGET))
        if t_g != t_o:
            continue
        dec.set_skip_mask(*mask); orc.set_skip_mask(*mask)
        last = t_o
        for _ in range(6):                                   # rounds of 3 draft steps and a verify, in lockstep
            pos0 = orc.positions()[0]                        # position of the row that starts the verify
            row, q_g, q_o, ok = [last], [], [], True
            for j in range(3):
                d_o = orc.draft_step(row[-1])
                d_g = dec.draft_step(row[-1])
                assert_logits_close(dec.get_last_logits(), orc.last()["logits"])
                qg, qo = check_draw(d_g, dec.get_last_logits()[0], orc.last()["logits"][0], d_o, oracle.uniform(seed, pos0 + 1 + j, oracle.DRAW_DRAFT))
                if d_g != d_o:
                    ok = False
                    break
                row.append(d_o); q_g.append(qg); q_o.append(qo)
            if not ok:
                break                                         # an undecided draw went the other way: this seed ends here
            a_o, out_o = orc.verify(row)
            p_o = [oracle.softmax_t(orc.last()["logits"][j], T) for j in range(len(row))]
            a_g, out_g = dec.verify(row)
            assert_logits_close(dec.get_last_logits(), orc.last()["logits"])
            p_g = [oracle.softmax_t(dec.get_last_logits()[j], T) for j in range(len(row))]
            rounds += 1
            if _verify_margin(p_g, q_g, row[1:], seed, pos0) > 1e-9:      # the rule on the GPU's own distributions
                a_r, out_r = oracle.spec_accept(np.array(p_g), np.array(q_g), row[1:], seed, pos0)
                assert (a_g, out_g.tolist()) == (a_r, out_r.tolist()), (seed, rounds)
                exact += 1
            if _verify_decided(p_o, q_o, p_g, q_g, row[1:], seed, pos0):
                assert (a_g, out_g.tolist()) == (a_o, out_o.tolist()), (seed, rounds)
                decided_rounds += 1
            if (a_g, out_g.tolist()) != (a_o, out_o.tolist()):
                break
            assert dec.positions() == orc.positions()
            last = int(out_o[-1])
    assert exact >= 20 and decided_draws >= 4 and decided_rounds >= 1, (exact, decided_draws, decided_rounds, rounds)


def test_cold_sampling_equals_greedy_and_identical_models_accept_everything(tiny_model, tiny_prompt):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    greedy, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_AR)
    cold, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_AR, temperature=1e-5, seed=5)
    assert cold.tolist() == greedy.tolist()                  # all mass on the argmax: the greedy loop
    cold_sp, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_SPEC, draft_len=4, m=2, n=1, temperature=1e-5, seed=5)
    assert cold_sp.tolist() == greedy.tolist()
    dec.set_skip_mask([0, 0, 0, 0], [0, 0, 0, 0])            # D = M: q = p, every draft is accepted
    a, st = dec.generate(tiny_prompt, 40, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=4, temperature=0.7, seed=9)
    assert st["accepted"] == st["drafted"] > 0
    dec.set_skip_mask([0, 0, 0, 0], [0, 0, 0, 0])
    b, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=4, temperature=0.7, seed=9)
    c, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_AR, temperature=0.7, seed=9)
    d, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_AR, temperature=0.7, seed=10)
    assert a.tolist() == b.tolist() and c.tolist() != d.tolist()       # reproducible, and the seed matters


def test_sampled_generation_equals_the_oracles_where_every_choice_is_decided(sharp_tiny, tiny_prompt):
    tiny_model = sharp_tiny
    # whole generations: compare token by token up to the first position where the oracle's choice was within MARGIN_U of
    # a threshold (found by replaying the oracle through its single steps is not needed: the oracle's own sequence decides)
    import paper_2410_01028_b200 as asd
    dec, orc = _pair(synth.TINY, tiny_model, max_seq=128)
    agree = 0
    for seed in range(6):
        ref, _, _ = orc.generate(tiny_prompt, 24, mode=oracle.MODE_AR, temperature=0.2, seed=seed)
        got, _ = dec.generate(tiny_prompt, 24, mode=asd.MODE_AR, temperature=0.2, seed=seed)
        n = next((i for i in range(24) if got[i] != ref[i]), 24)
        agree += n
        if n < 24:                                            # the first difference must be an undecided draw of the oracle
            orc.reset(); orc.set_sampling(0.2, seed)
            t = orc.prefill(tiny_prompt)
            for i in range(1, n + 1):
                t = orc.decode_step(int(ref[i - 1]))
            probs = oracle.softmax_t(orc.last()["logits"][-1], 0.2)
            tok, margin = _draw_margin(probs, oracle.uniform(seed, len(tiny_prompt) + n, oracle.DRAW_TARGET))
            # ... within what a logit error at the tolerance can move a cumulative probability at this temperature
            # (|dp| <= p |dl| / T summed over the vocabulary: 2 * 2e-2 * max|logit| / T is far above anything seen; 5e-2 is used)
            assert tok == ref[n] and margin <= 5e-2, (seed, n, margin)
    assert agree >= 6 * 12


def test_verify_with_sampling_refuses_tokens_it_did_not_draft(tiny_model, tiny_prompt):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    dec.set_sampling(0.9, 1)
    t = dec.prefill(tiny_prompt)
    with pytest.raises(asd.AsdError) as e:
        dec.verify([t, 4, 5])
    assert e.value.code == asd.binding.ERR_STATE
    d = dec.draft_step(t)
    a, out = dec.verify([t, d])
    assert 0 <= a <= 1 and len(out) == a + 1
    with pytest.raises(asd.AsdError) as e:
        dec.set_sampling(-1.0, 0)
    assert e.value.code == asd.binding.ERR_ARG
    dec.set_sampling(0.0)                                     # back to greedy on the same context
    dec.reset()
    assert isinstance(dec.prefill(tiny_prompt), int)
