"""Comparison helpers shared by the GPU parity tests (tolerances of the parity contract)."""
import collections

import numpy as np

# soft = token mismatches at steps whose top-2 logit gap in the oracle is at most MARGIN (allowed);
# decided = steps whose gap exceeds MARGIN, where the GPU's token had to equal the oracle's (and did)
Compare = collections.namedtuple("Compare", "soft decided")

LOGIT_TOL = 2e-2     # |l_gpu - l_orc| <= LOGIT_TOL * max|l_orc| per row
COS_TOL = 1e-3       # absolute, per sublayer and row
MARGIN = 1e-2        # token ids must agree wherever the oracle's top-2 logit gap exceeds this
MASK_MARGIN = 1e-3   # skip masks must agree wherever |C_l - alpha| exceeds this


def assert_logits_close(gpu, orc):
    tol = LOGIT_TOL * np.abs(orc).max(axis=-1, keepdims=True)
    err = np.abs(gpu - orc)
    assert np.all(err <= tol), f"logit error {err.max():.4g} above tolerance {tol.min():.4g}"


def assert_cos_close(gpu, orc):
    assert gpu.shape == orc.shape
    both_nan = np.isnan(gpu) & np.isnan(orc)
    assert np.array_equal(np.isnan(gpu), np.isnan(orc)), "skipped sublayers differ"
    err = np.abs(np.where(both_nan, 0, gpu) - np.where(both_nan, 0, orc))
    assert err.max() <= COS_TOL, f"cosine error {err.max():.3g}"


def teacher_forced_compare(dec, orc, prompt, max_new, check_logits=True):
    """Feed the oracle's greedy tokens through the GPU decoder step by step.

    At every step the GPU's argmax must equal the oracle's wherever the oracle's top-2 margin exceeds MARGIN;
    logits and per-sublayer cosines are compared at every step.  Returns Compare(soft, decided); at least one step
    must have been decided, so that the token comparison cannot pass vacuously.
    """
    ref, margins, _ = orc.generate(prompt, max_new)
    orc.reset()
    dec.reset()
    if check_logits:
        dec.set_debug(True)
    t_o = orc.prefill(prompt)
    t_g = dec.prefill(prompt)
    soft = decided = 0

    def check(tok_g, tok_o, margin, step):
        nonlocal soft, decided
        if margin > MARGIN:
            assert tok_g == tok_o, f"token mismatch at step {step} with margin {margin}"
            decided += 1
        elif tok_g != tok_o:
            soft += 1

    assert t_o == ref[0]
    check(t_g, t_o, margins[0], 0)
    for i in range(1, max_new):
        o = orc.decode_step(int(ref[i - 1]))
        g = dec.decode_step(int(ref[i - 1]))
        assert o == ref[i]
        check(g, o, margins[i], i)
        last = orc.last()
        ca, cm = dec.get_last_cosines()
        assert_cos_close(ca, last["cos_attn"])
        assert_cos_close(cm, last["cos_mlp"])
        if check_logits:
            assert_logits_close(dec.get_last_logits(), last["logits"])
    assert decided > 0, "no step had a top-2 logit gap above the margin: the token comparison decided nothing"
    return Compare(soft, decided)


def verify_outcomes_agree(a_g, out_g, a_o, out_o, margins):
    """Greedy acceptance of one verify pass, GPU against oracle.

    The oracle's outcome (a_o accepted drafts, then M's own token) is decided by its rows 0..a_o. Where every one of
    those rows has a top-2 logit gap above MARGIN the GPU must report the same acceptance and the same tokens; the
    function then returns 1 (a decided comparison), otherwise 0.
    """
    if np.all(np.asarray(margins)[: a_o + 1] > MARGIN):
        assert a_g == a_o and list(out_g) == list(out_o), (a_g, list(out_g), a_o, list(out_o))
        return 1
    return 0


def argmax_rows_agree(gpu_logits, orc_last, rows=None):
    """Token ids of the rows of one pass: the argmax of the GPU's logits must equal the oracle's argmax in every row
    whose top-2 gap in the oracle exceeds MARGIN. Returns how many rows were decided that way."""
    margin, am = np.asarray(orc_last["margin"]), np.asarray(orc_last["argmax"])
    if rows is not None:
        margin, am = margin[rows], am[rows]
    got = np.argmax(gpu_logits, axis=-1)
    assert got.shape == am.shape
    decided = margin > MARGIN
    assert np.array_equal(got[decided], am[decided]), (got, am, margin)
    return int(decided.sum())
