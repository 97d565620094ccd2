"""Draft exiting: a round stops drafting after the first draft token whose top-2 logit gap in the draft model is below
a threshold (the fixed-threshold form of the mechanism the paper's Section 4 takes from Draft & Verify).

CPU part: pins of the oracle (the gap against a sort of the logits; the loop against a step-by-step replay; limiting
thresholds; losslessness). GPU part: the library's gaps against its own logits and the oracle's, its loop against a
step-by-step replay through the single-step calls.
"""
import numpy as np
import pytest

import oracle
import synth
from helpers import LOGIT_TOL

SMALL = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)


@pytest.fixture(scope="module")
def small():
    return synth.make_model(SMALL, seed=7, std=0.2)


def _gap_by_sorting(logits):
    s = np.sort(logits.astype(np.float32), axis=-1)
    return s[..., -1] - s[..., -2]


def _replay(dec, mask, prompt, max_new, k_max, thr, gap_of_last_pass):
    """The speculative loop written with the single-step calls; returns (tokens, rounds, drafted, accepted)."""
    dec.reset()
    dec.set_skip_mask(*mask)  # a reset clears the mask
    out = [dec.prefill(prompt)]
    rounds = drafted = accepted = 0
    while len(out) < max_new:
        k = min(k_max, max_new - len(out) - 1)
        row = [out[-1]]
        for j in range(k):
            row.append(dec.draft_step(row[-1]))
            if thr > 0 and j + 1 < k and gap_of_last_pass(dec) < np.float32(thr):
                break
        a, toks = dec.verify(np.array(row, np.int32))
        rounds += 1
        drafted += len(row) - 1
        accepted += a
        out.extend(int(t) for t in toks)
    return out[:max_new], rounds, drafted, accepted


def test_oracle_gap_is_top1_minus_top2(small):
    o = oracle.Oracle(small, max_seq=32)
    o.prefill(synth.make_prompt(SMALL.vocab, 9, seed=31))
    last = o.last()
    np.testing.assert_array_equal(last["margin"], _gap_by_sorting(last["logits"]))


@pytest.mark.parametrize("thr", [0.05, 0.3, 1.0])
def test_oracle_loop_equals_step_by_step_replay(small, thr):
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=32)
    o = oracle.Oracle(small, max_seq=64)
    ar, _, _ = o.generate(prompt, 24, mode=oracle.MODE_AR)
    o.set_skip_mask([0, 1], [1, 0])
    toks, _, st = o.generate(prompt, 24, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=5, draft_exit_margin=thr)
    assert toks.tolist() == ar.tolist()  # lossless whatever the threshold
    r_toks, rounds, drafted, accepted = _replay(o, ([0, 1], [1, 0]), prompt, 24, 5, thr, lambda d: d.last()["margin"][0])
    assert r_toks == ar.tolist()
    assert (st["rounds"], st["drafted"], st["accepted"]) == (rounds, drafted, accepted)


def test_oracle_limiting_thresholds(small):
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=33)
    o = oracle.Oracle(small, max_seq=64)
    o.set_skip_mask([1, 0], [0, 1])
    _, _, base = o.generate(prompt, 20, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4)
    o.set_skip_mask([1, 0], [0, 1])
    _, _, off = o.generate(prompt, 20, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4, draft_exit_margin=0.0)
    o.set_skip_mask([1, 0], [0, 1])
    _, _, one = o.generate(prompt, 20, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=1)
    o.set_skip_mask([1, 0], [0, 1])
    _, _, huge = o.generate(prompt, 20, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4, draft_exit_margin=1e30)
    key = lambda s: (s["rounds"], s["drafted"], s["accepted"])
    assert key(off) == key(base)   # threshold 0: every round drafts draft_len tokens
    assert key(huge) == key(one)   # a threshold nothing reaches: one draft per round
    assert huge["rounds"] - 1 <= huge["drafted"] <= huge["rounds"]  # the last round may have no token left to draft


# ------------------------------------------------------------------ the library
@pytest.fixture(scope="module")
def tiny_dec(tiny_model):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    yield dec
    dec.close()


@pytest.mark.gpu
def test_gpu_gap_equals_its_own_logits_and_the_oracles(tiny_dec, tiny_model, tiny_prompt):
    dec = tiny_dec
    orc = oracle.Oracle(tiny_model, max_seq=128)
    dec.reset()
    dec.set_debug(True)
    t_g, t_o = dec.prefill(tiny_prompt[:16]), orc.prefill(tiny_prompt[:16])  # short prompt: row passes, all rows kept

    def check():
        gaps, logits, ref = dec.get_last_margins(), dec.get_last_logits(), orc.last()
        assert gaps.shape == (logits.shape[0],)
        np.testing.assert_array_equal(gaps, _gap_by_sorting(logits))  # exactly the gap of the logits it computed
        tol = 2 * LOGIT_TOL * np.abs(ref["logits"]).max(axis=-1)
        assert np.all(np.abs(gaps - ref["margin"][-gaps.size:]) <= tol[-gaps.size:])

    check()
    dec.decode_step(t_o); orc.decode_step(t_o)
    check()
    row = np.array([int(orc.last()["argmax"][0]), 3, 5, 7, 11], np.int32)
    dec.verify(row); orc.verify(row)
    check()
    dec.set_debug(False)


@pytest.mark.gpu
@pytest.mark.parametrize("thr", [0.0, 0.02, 0.1, 1e30])
def test_gpu_loop_equals_step_by_step_replay(tiny_dec, tiny_prompt, thr):
    import paper_2410_01028_b200 as asd
    dec = tiny_dec
    ar, _ = dec.generate(tiny_prompt, 40, mode=asd.MODE_AR)
    mask_a, mask_m = [0, 1, 0, 0], [0, 0, 1, 0]
    dec.set_skip_mask(mask_a, mask_m)
    sp, st = dec.generate(tiny_prompt, 40, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=5, draft_exit_margin=thr)
    assert sp.tolist() == ar.tolist()
    toks, rounds, drafted, accepted = _replay(dec, (mask_a, mask_m), tiny_prompt, 40, 5, thr, lambda d: d.get_last_margins()[0])
    assert toks == ar.tolist()
    assert (st["rounds"], st["drafted"], st["accepted"]) == (rounds, drafted, accepted)
    if thr >= 1e30:
        assert rounds - 1 <= drafted <= rounds  # the last round may have no token left to draft
