"""GPU parity at the widths, launch shapes and context lengths of the benchmark configurations.

The oracle cannot run a whole 32-layer model for hundreds of positions in seconds, so the full-size checks are
(a) element-wise parity on models with the FULL widths (7B and 13B rows, vocabulary, head size: the same grid,
shared-memory plan, ring and window sizes as the benchmark) but few layers and short prompts, which the oracle
finishes in seconds; (b) a long-prompt case in which every CTA owns several attention work items; and
(c) properties that hold at any size on the full 32-layer 7B-shaped model in the configuration bench.py times.
"""
import dataclasses

import numpy as np
import pytest

import oracle
import synth
from helpers import COS_TOL, teacher_forced_compare, verify_outcomes_agree

pytestmark = pytest.mark.gpu


def _pair(shape, max_seq, seed=0):
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=seed)
    dec = asd.Decoder(shape, max_seq=max_seq, max_draft=8)
    dec.load_weights_host(model)
    return model, dec, oracle.Oracle(model, max_seq=max_seq)


@pytest.mark.parametrize("base,layers,S,new,mode", [(synth.LLAMA_7B, 2, 43, 6, "gemm"), (synth.LLAMA_7B, 2, 43, 6, "rows"),
                                                    (synth.LLAMA_13B, 1, 21, 4, "rows"), (synth.LLAMA_13B, 1, 37, 4, "gemm")])
def test_full_width_few_layers_teacher_forced(base, layers, S, new, mode):
    import paper_2410_01028_b200 as asd
    shape = dataclasses.replace(base, n_layers=layers)
    _, dec, orc = _pair(shape, max_seq=S + new + 16)
    dec.set_prefill_mode(asd.PREFILL_GEMM if mode == "gemm" else asd.PREFILL_ROWS)   # both prompt paths at full width
    prompt = synth.make_prompt(shape.vocab, S, seed=1)
    teacher_forced_compare(dec, orc, prompt, new)
    ca_g, cm_g, _ = dec.get_similarity()
    ca_o, cm_o, _ = orc.similarity()
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL


def test_full_width_verify_rows_match_oracle_and_decode():
    import paper_2410_01028_b200 as asd
    shape = dataclasses.replace(synth.LLAMA_7B, n_layers=2)
    _, dec, orc = _pair(shape, max_seq=64)
    prompt = synth.make_prompt(shape.vocab, 19, seed=2)
    ref, margins, _ = orc.generate(prompt, 10)
    decided = 0
    for k in (4, 8):
        orc.reset(); dec.reset()
        t = orc.prefill(prompt); dec.prefill(prompt)
        row = np.concatenate([[t], ref[1:k + 1]])
        row[-1] = (row[-1] + 1) % shape.vocab          # the last draft is wrong: k-1 drafts accepted
        a_o, out_o = orc.verify(row)
        m = orc.last()["margin"]
        dec.set_debug(True)
        a_g, out_g = dec.verify(row)
        from helpers import assert_cos_close, assert_logits_close
        assert_logits_close(dec.get_last_logits(), orc.last()["logits"])
        # top-2 logit gap of every row (what draft exiting looks at): exactly the gap of the logits the pass computed,
        # across all CTAs' partial results, and the oracle's within the logit tolerance
        gl = np.sort(dec.get_last_logits(), axis=-1)
        np.testing.assert_array_equal(dec.get_last_margins(), gl[:, -1] - gl[:, -2])
        assert np.all(np.abs(dec.get_last_margins() - m) <= 2 * 2e-2 * np.abs(orc.last()["logits"]).max(axis=-1))
        ca, cm = dec.get_last_cosines()
        assert_cos_close(ca, orc.last()["cos_attn"]); assert_cos_close(cm, orc.last()["cos_mlp"])
        assert a_o == k - 1
        decided += verify_outcomes_agree(a_g, out_g, a_o, out_o, m)
    assert decided >= 1                                   # acceptance and tokens were compared at full width
    ar, _ = dec.generate(prompt, 24, mode=asd.MODE_AR)
    for k in (1, 4, 6, 8):
        dec.set_skip_mask([0, 1], [1, 0])
        sp, _ = dec.generate(prompt, 24, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=k)
        assert sp.tolist() == ar.tolist(), k


def test_long_prompt_several_attention_items_per_cta():
    # 16 heads x 11 chunks of 128 keys = 176 attention work items for 148 CTAs, prompt crossing many chunk borders
    shape = synth.DecoderShape(n_layers=2, d_model=1024, n_heads=16, head_dim=64, d_ffn=2752, vocab=5003)
    _, dec, orc = _pair(shape, max_seq=1400)
    prompt = synth.make_prompt(shape.vocab, 1300, seed=3)
    teacher_forced_compare(dec, orc, prompt, 5)
    ca_g, _, n = dec.get_similarity()
    ca_o, _, _ = orc.similarity()
    assert n == 1300 and np.abs(ca_g - ca_o).max() <= COS_TOL


def test_7b_shaped_model_properties_in_the_benchmark_configuration():
    import paper_2410_01028_b200 as asd
    shape = synth.LLAMA_7B
    model = synth.make_model(shape, seed=0)
    dec = asd.Decoder(shape, max_seq=512 + 64 + 16, max_draft=8)
    dec.load_weights_host(model)
    prompt = synth.make_prompt(shape.vocab, 512, seed=1)
    new = 48
    ar, st_ar = dec.generate(prompt, new, mode=asd.MODE_AR)
    assert st_ar["full_passes"] == new - 1 and st_ar["prefill_rows"] == 512
    ca, cm, n = dec.get_similarity()
    assert n == 512 and np.all(np.abs(ca) <= 1 + 1e-6) and np.all(np.abs(cm) <= 1 + 1e-6)
    assert ca[0] < 0.5 and np.median(ca) > 0.98          # the recipe's similarity profile (first layer far from 1)
    for kw in (dict(alpha=0.9997, flags=asd.USE_CS | asd.USE_RULE2, draft_len=4, draft_exit_margin=0.1),  # bench.py's default
               dict(alpha=0.9995, flags=asd.USE_CS | asd.USE_RULE2, draft_len=4),
               dict(alpha=0.985, m=3, n=2, flags=asd.ADMG_ALL, draft_len=6)):           # Table 2's hyper-parameters
        sp, st = dec.generate(prompt, new, mode=asd.MODE_SPEC, **kw)
        assert sp.tolist() == ar.tolist()                 # lossless, bit for bit
        assert st["accepted"] + st["rounds"] == new - 1 and 0 <= st["accepted"] <= st["drafted"]
        skip_a, skip_m = dec.admg_update(kw["alpha"], kw.get("m", 3), kw.get("n", 2), kw["flags"])
        ra, rm = oracle.admg(ca, kw["alpha"], kw.get("m", 3), kw.get("n", 2), kw["flags"])
        assert skip_a.tolist() == ra.tolist() and skip_m.tolist() == rm.tolist()
        assert st["bytes_draft"] / max(st["draft_passes"], 1) < st_ar["bytes_full"] / st_ar["full_passes"]
    # paper defaults: rule 1 removes every third MLP below the last two layers -> 10 MLPs, 10 + CS attention layers
    assert int(skip_m.sum()) == 10 and int(skip_a.sum()) >= 10
    # sampled element-wise check against the oracle at full depth: first 6 prompt rows (the oracle's cost is per row)
    orc = oracle.Oracle(model, max_seq=16)
    dec.reset()
    dec.set_debug(True)
    t_g, t_o = dec.prefill(prompt[:6]), orc.prefill(prompt[:6])
    from helpers import assert_cos_close, assert_logits_close
    assert_logits_close(dec.get_last_logits(), orc.last()["logits"])
    ca_g, cm_g = dec.get_last_cosines()
    assert_cos_close(ca_g, orc.last()["cos_attn"]); assert_cos_close(cm_g, orc.last()["cos_mlp"])
    from helpers import argmax_rows_agree
    assert argmax_rows_agree(dec.get_last_logits(), orc.last()) >= 3      # token ids of the six rows at full depth
    assert t_g == int(np.argmax(dec.get_last_logits()[-1]))
