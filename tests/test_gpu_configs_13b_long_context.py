"""GPU parity on the two benchmark configurations that stress what the small cases do not.

* The 13B-shaped decoder with draft length 6: full width (d = 5120, ffn = 13824, 40 heads, vocabulary 32000), two
  layers, a seven-row verify pass against the oracle (logits, cosines, acceptance) and speculative == autoregressive
  output for k = 6, through both prompt paths.
* The long-context decoder: more than 8192 cached positions at head size 128, so that every head has 65 attention
  chunks, the chunk merge runs over several batches, the dense prompt path takes five chunks of 2048 rows and a
  generation crosses the chunk border at position 8192. Two layers and a narrow model keep the oracle's quadratic
  prompt pass within about a minute.
"""
import dataclasses

import numpy as np
import pytest

import oracle
import synth
from helpers import (COS_TOL, argmax_rows_agree, assert_cos_close, assert_logits_close, teacher_forced_compare,
                     verify_outcomes_agree)

pytestmark = pytest.mark.gpu


def _pair(shape, max_seq, seed=0, std=0.02):
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=seed, std=std)
    dec = asd.Decoder(shape, max_seq=max_seq, max_draft=8)
    dec.load_weights_host(model)
    return model, dec, oracle.Oracle(model, max_seq=max_seq)


def _kv_rows_close(dec, orc, layer, positions):
    """bf16 K/V rows: one ulp of the value; below the first layer also 1e-2 of the row's scale (inherited flips)."""
    for p in positions:
        kg, vg = dec.get_kv(layer, p)
        ko, vo = orc.kv(layer, p)
        for g, o in ((synth.bf16_to_f32(kg), ko), (synth.bf16_to_f32(vg), vo)):
            assert np.all(np.abs(g - o) <= 2 ** -7 * np.abs(o) + (0.0 if layer == 0 else 1e-2) * np.abs(o).max()), (layer, p)


def _verify_against_oracle(dec, orc, row):
    """One verify pass of len(row) rows on both sides: logits, cosines, acceptance. Returns (decided, a, out)."""
    a_o, out_o = orc.verify(row)
    last = orc.last()
    a_g, out_g = dec.verify(row)
    assert_logits_close(dec.get_last_logits(), last["logits"])
    ca, cm = dec.get_last_cosines()
    assert_cos_close(ca, last["cos_attn"])
    assert_cos_close(cm, last["cos_mlp"])
    rows_decided = argmax_rows_agree(dec.get_last_logits(), last)
    decided = verify_outcomes_agree(a_g, out_g, a_o, out_o, last["margin"])
    assert dec.positions() == orc.positions() or not decided
    return decided, rows_decided, a_o, out_o


# ------------------------------------------------------------------ 13B shape, draft length 6
@pytest.mark.parametrize("mode", ["gemm", "rows"])
def test_13b_width_two_layers_seven_row_verify_and_lossless_generation(mode):
    import paper_2410_01028_b200 as asd
    shape = dataclasses.replace(synth.LLAMA_13B, n_layers=2)
    S, k = 41, 6
    _, dec, orc = _pair(shape, max_seq=S + 64)
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_GEMM if mode == "gemm" else asd.PREFILL_ROWS)
    prompt = synth.make_prompt(shape.vocab, S, seed=4)
    ref, _, _ = orc.generate(prompt, 16)                 # the oracle's greedy continuation: the drafts fed below
    orc.reset()
    t_o, t_g = orc.prefill(prompt), dec.prefill(prompt)
    assert t_o == ref[0]
    ca_g, cm_g, n_g = dec.get_similarity()
    ca_o, cm_o, n_o = orc.similarity()
    assert n_g == n_o == S
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    # seven rows, every draft right: six accepted plus the model's own next token
    d1, r1, a, out = _verify_against_oracle(dec, orc, np.concatenate([[t_o], ref[1:k + 1]]))
    assert a == k and out.tolist() == ref[1:k + 2].tolist()
    # seven rows, the fourth draft wrong: three accepted, the model's token replaces the fourth
    n0 = 1 + k + 1
    row = np.concatenate([[ref[n0 - 1]], ref[n0:n0 + k]])
    row[4] = (row[4] + 1) % shape.vocab
    d2, r2, a, out = _verify_against_oracle(dec, orc, row)
    assert a == 3 and out.tolist() == ref[n0:n0 + 4].tolist()
    assert d1 + d2 >= 1 and r1 + r2 >= 7                 # acceptance and token ids were decided, not skipped
    # lossless: speculative output equals autoregressive output bit for bit at draft length 6 (and around it)
    ar, _ = dec.generate(prompt, 30, mode=asd.MODE_AR)
    for kk, mask in ((6, ([0, 1], [1, 0])), (6, ([1, 0], [0, 0])), (5, ([1, 1], [1, 1])), (7, ([0, 0], [0, 0]))):
        dec.set_skip_mask(*mask)
        sp, st = dec.generate(prompt, 30, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=kk)
        assert sp.tolist() == ar.tolist(), (kk, mask)
        assert st["accepted"] + st["rounds"] == 29
    assert st["accepted"] == st["drafted"]               # empty mask: the draft is the full model


# ------------------------------------------------------------------ more than 8192 cached positions
LONG = synth.DecoderShape(n_layers=2, d_model=512, n_heads=4, head_dim=128, d_ffn=256, vocab=2003)


def test_long_context_beyond_8192_positions():
    import paper_2410_01028_b200 as asd
    S = 8200                                             # 4 dense chunks of 2048 rows + 7 rows + the last row; 65 chunks of 128 keys
    model, dec, orc = _pair(LONG, max_seq=S + 64, seed=5, std=0.05)
    prompt = synth.make_prompt(LONG.vocab, S, seed=6)
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_GEMM)
    # the lossless property first, where the generation crosses the chunk border at position 8192 (prompt of 8185)
    ar, st_ar = dec.generate(prompt[:8185], 28, mode=asd.MODE_AR)
    assert st_ar["prefill_rows"] == 8185
    for k, mask in ((4, ([0, 1], [0, 0])), (8, ([1, 0], [0, 1])), (8, ([0, 0], [0, 0]))):
        dec.set_skip_mask(*mask)
        sp, st = dec.generate(prompt[:8185], 28, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=k)
        assert sp.tolist() == ar.tolist(), (k, mask)
    assert st["accepted"] == st["drafted"] > 0
    # the same continuation with the prompt fed through the row passes (16 rows at a time through the pass kernel)
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    dec.generate(prompt[:8185], 2, mode=asd.MODE_AR)
    ca_r, cm_r, _ = dec.get_similarity()
    dec.set_prefill_mode(asd.PREFILL_GEMM)

    # now against the oracle: the whole prompt, then verify passes and decode steps on top of 8200 cached positions
    dec.reset()
    t_g, t_o = dec.prefill(prompt), orc.prefill(prompt)
    last = orc.last()
    assert_logits_close(dec.get_last_logits(), last["logits"][-1:])
    decided = argmax_rows_agree(dec.get_last_logits(), last, slice(-1, None))
    ca_g, cm_g, n_g = dec.get_similarity()
    ca_o, cm_o, n_o = orc.similarity()
    assert n_g == n_o == S
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    # (the row-pass prompt above was 15 rows shorter: its mean similarities agree to well within the tolerance too)
    assert np.abs(ca_r - ca_o).max() <= 2 * COS_TOL and np.abs(cm_r - cm_o).max() <= 2 * COS_TOL
    for layer in range(LONG.n_layers):
        _kv_rows_close(dec, orc, layer, (0, 127, 128, 2047, 2048, 4095, 4096, 6143, 6144, 8191, 8192, S - 1))
    # drafts = the GPU's own greedy continuation of the full prompt (the oracle decides what it accepts)
    cont, _ = dec.generate(prompt, 24, mode=asd.MODE_AR)
    dec.reset()
    dec.prefill(prompt)
    assert cont[0] == t_g
    # five rows at positions 8200..8204
    d1, r1, a1, out1 = _verify_against_oracle(dec, orc, np.concatenate([[t_o], cont[1:5]]))
    # nine rows on top of what was committed, the last draft wrong
    n0 = 1 + a1 + 1
    row = np.concatenate([[out1[-1]], cont[n0:n0 + 8]])
    row[-1] = (row[-1] + 1) % LONG.vocab
    d2, r2, a2, out2 = _verify_against_oracle(dec, orc, row)
    assert d1 + d2 >= 1 and r1 + r2 >= 7
    assert a1 + a2 >= 6                                  # most of the right drafts were accepted by both sides
    # teacher-forced one-row passes from there
    t = int(out2[-1])
    for _ in range(3):
        o, g = orc.decode_step(t), dec.decode_step(t)
        assert_logits_close(dec.get_last_logits(), orc.last()["logits"])
        ca, cm = dec.get_last_cosines()
        assert_cos_close(ca, orc.last()["cos_attn"]); assert_cos_close(cm, orc.last()["cos_mlp"])
        decided += argmax_rows_agree(dec.get_last_logits(), orc.last())
        assert g == int(np.argmax(dec.get_last_logits()[0]))
        t = o
    assert decided >= 2
