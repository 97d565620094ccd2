"""GPU edge cases of the decoding loops against the oracle: the degenerate sizes of the method (one-token prompt, one
generated token, draft length 0, end-of-sequence inside an accepted run, a cache filled to its last position)."""
import numpy as np
import pytest

import oracle
import synth

pytestmark = pytest.mark.gpu

SMALL = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)


@pytest.fixture(scope="module")
def pair():
    import paper_2410_01028_b200 as asd
    model = synth.make_model(SMALL, seed=7, std=0.2)
    dec = asd.Decoder(SMALL, max_seq=48, max_draft=8)
    dec.load_weights_host(model)
    return dec, oracle.Oracle(model, max_seq=48)


def _same_where_decided(got, ref, margins):
    first_soft = next((i for i in range(len(ref)) if margins[i] <= 1e-2), len(ref))
    assert list(got[:first_soft]) == list(ref[:first_soft])
    return first_soft


def test_one_token_prompt_and_one_generated_token(pair):
    import paper_2410_01028_b200 as asd
    dec, orc = pair
    ref, margins, _ = orc.generate([7], 12)
    for mode, kw in ((asd.MODE_AR, {}), (asd.MODE_SPEC_MANUAL_MASK, dict(draft_len=4))):
        dec.set_skip_mask([0, 1], [1, 0])
        got, st = dec.generate([7], 12, mode=mode, **kw)
        assert _same_where_decided(got, ref, margins) >= 6
        assert st["prefill_rows"] == 1 and dec.positions()[0] == 1 + 11
    # a single new token is the prompt pass's own token: no decode, draft or verify pass runs
    for mode in (asd.MODE_AR, asd.MODE_SPEC):
        got, st = dec.generate([7, 8, 9], 1, mode=mode, draft_len=4)
        ref1, m1, _ = orc.generate([7, 8, 9], 1)
        assert len(got) == 1 and (m1[0] <= 1e-2 or got[0] == ref1[0])
        assert st["full_passes"] == st["draft_passes"] == st["verify_passes"] == 0


def test_draft_length_zero_is_autoregressive_decoding_through_verify_passes(pair):
    import paper_2410_01028_b200 as asd
    dec, orc = pair
    prompt = synth.make_prompt(SMALL.vocab, 5, seed=3)
    ar, _ = dec.generate(prompt, 16, mode=asd.MODE_AR)
    dec.set_skip_mask([1, 1], [1, 1])
    sp, st = dec.generate(prompt, 16, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=0)
    assert sp.tolist() == ar.tolist()
    assert st["draft_passes"] == 0 and st["verify_passes"] == 15 and st["drafted"] == 0 and st["accepted"] == 0
    dec.reset()
    t = dec.prefill(prompt)
    a, out = dec.verify([t])                                   # k = 0: one row, nothing to accept, M's own token comes back
    assert a == 0 and out.tolist() == [ar[1]]


def test_end_of_sequence_stops_inside_an_accepted_run(pair):
    import paper_2410_01028_b200 as asd
    dec, orc = pair
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=4)
    ar, _ = dec.generate(prompt, 20, mode=asd.MODE_AR)
    eos = int(ar[7])
    stop = ar.tolist().index(eos) + 1                           # the first occurrence ends the output, the token included
    got_ar, _ = dec.generate(prompt, 20, mode=asd.MODE_AR, eos_id=eos)
    assert got_ar.tolist() == ar[:stop].tolist()
    dec.set_skip_mask([0, 0], [0, 0])                           # D = M: every draft accepted, so the eos sits inside a run
    got_sp, _ = dec.generate(prompt, 20, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=5, eos_id=eos)
    assert got_sp.tolist() == ar[:stop].tolist()
    ref, _, _ = orc.generate(prompt, 20, mode=oracle.MODE_AR, eos_id=eos)
    ref_full, margins, _ = orc.generate(prompt, 20, mode=oracle.MODE_AR)
    if np.all(margins[:len(ref)] > 1e-2) and list(ref_full[:stop]) == ar[:stop].tolist():
        assert got_ar.tolist() == ref.tolist()


def test_cache_filled_to_its_last_position(pair):
    import paper_2410_01028_b200 as asd
    dec, orc = pair
    prompt = synth.make_prompt(SMALL.vocab, 30, seed=5)
    # 30 prompt positions + 18 committed tokens = max_seq 48: the last rounds must shrink their draft length
    ar, _ = dec.generate(prompt, 19, mode=asd.MODE_AR)
    assert dec.positions()[0] == 48
    for k in (3, 8):
        dec.set_skip_mask([0, 1], [0, 0])
        sp, st = dec.generate(prompt, 19, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=k)
        assert sp.tolist() == ar.tolist() and dec.positions()[0] == 48
    with pytest.raises(asd.AsdError) as e:
        dec.decode_step(int(ar[-1]))                             # one position too many
    assert e.value.code == asd.binding.ERR_OVERFLOW
    with pytest.raises(asd.AsdError) as e:
        dec.generate(prompt, 49, mode=asd.MODE_AR)
    assert e.value.code == asd.binding.ERR_OVERFLOW
