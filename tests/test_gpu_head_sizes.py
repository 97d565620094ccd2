"""Head sizes at the ends of what the pass kernel supports: 32 (a K/V box narrower than 128 bytes: no swizzle) and 256
(four 64-column boxes per key row, two query elements per thread in the tagged handoff). Teacher-forced parity with the
oracle, speculative == autoregressive, and row m of a verify pass bit-identical to a one-row pass."""
import numpy as np
import pytest

import oracle
import synth
from helpers import COS_TOL, teacher_forced_compare

pytestmark = pytest.mark.gpu

HD256 = synth.DecoderShape(n_layers=2, d_model=512, n_heads=2, head_dim=256, d_ffn=1024, vocab=997)
HD32 = synth.DecoderShape(n_layers=2, d_model=256, n_heads=8, head_dim=32, d_ffn=512, vocab=613, n_kv_heads=4)


@pytest.mark.parametrize("shape", [HD256, HD32], ids=["hd256", "hd32_gqa"])
def test_head_size_against_oracle_and_row_invariance(shape):
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=5, std=0.05)
    dec = asd.Decoder(shape, max_seq=320, max_draft=8)
    dec.load_weights_host(model)
    orc = oracle.Oracle(model, max_seq=320)
    prompt = synth.make_prompt(shape.vocab, 140, seed=6)          # two 128-key chunks per head
    teacher_forced_compare(dec, orc, prompt, 16)
    ca_g, cm_g, _ = dec.get_similarity()
    ca_o, cm_o, _ = orc.similarity()
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    # lossless
    ar, _ = dec.generate(prompt, 24, mode=asd.MODE_AR)
    for k in (1, 4, 8):
        dec.set_skip_mask(np.array([0, 1]), np.array([1, 0]))
        sp, _ = dec.generate(prompt, 24, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=k)
        assert sp.tolist() == ar.tolist(), k
    # row invariance: five rows against five one-row passes
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    cont = synth.make_prompt(shape.vocab, 4, seed=7)
    dec.reset()
    t = dec.prefill(prompt)
    rows = [int(t)] + [int(v) for v in cont]
    one = []
    for r in rows:
        dec.decode_step(r)
        one.append(dec.get_last_logits()[0].copy())
    dec.reset()
    dec.prefill(prompt)
    dec.verify(rows)
    lg = dec.get_last_logits()
    for m in range(5):
        np.testing.assert_array_equal(lg[m], one[m])


WIDE = synth.DecoderShape(n_layers=1, d_model=6144, n_heads=48, head_dim=128, d_ffn=2048, vocab=509)


def test_rows_longer_than_the_register_paths_hold(request):
    """d_model above 5760: the RMSNorm stages take the general (strided) path and the one-row pass synchronises at the
    grid barrier (the tagged handoff needs its three chunks per thread). Against the oracle, lossless, row-invariant."""
    import paper_2410_01028_b200 as asd
    model = synth.make_model(WIDE, seed=8, std=0.02)
    dec = asd.Decoder(WIDE, max_seq=96, max_draft=8)
    dec.load_weights_host(model)
    orc = oracle.Oracle(model, max_seq=96)
    prompt = synth.make_prompt(WIDE.vocab, 40, seed=9)
    teacher_forced_compare(dec, orc, prompt, 8)
    ar, _ = dec.generate(prompt, 16, mode=asd.MODE_AR)
    for k in (2, 5):
        dec.set_skip_mask(np.array([0]), np.array([0]))
        sp, _ = dec.generate(prompt, 16, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=k)
        assert sp.tolist() == ar.tolist(), k
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    cont = synth.make_prompt(WIDE.vocab, 2, seed=10)
    dec.reset()
    t = dec.prefill(prompt)
    rows = [int(t)] + [int(v) for v in cont]
    one = []
    for r in rows:
        dec.decode_step(r)
        one.append(dec.get_last_logits()[0].copy())
    dec.reset()
    dec.prefill(prompt)
    dec.verify(rows)
    lg = dec.get_last_logits()
    for m in range(3):
        np.testing.assert_array_equal(lg[m], one[m])
