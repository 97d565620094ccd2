"""Comparison helpers shared by the GPU parity tests (tolerances of the parity contract)."""
import numpy as np

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
    logits and per-sublayer cosines are compared at every step.  Returns the number of low-margin mismatches.
    """
    ref, margins, _ = orc.generate(prompt, max_new)
    orc.reset()
    dec.reset()
    if check_logits:
        dec.set_debug(True)
    t_o = orc.prefill(prompt)
    t_g = dec.prefill(prompt)
    soft = 0

    def check(tok_g, tok_o, margin, step):
        nonlocal soft
        if tok_g != tok_o:
            assert margin <= MARGIN, f"token mismatch at step {step} with margin {margin}"
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
    return soft
