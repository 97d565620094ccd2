"""Row m of an M-row pass equals a one-row pass at the same position bit for bit, for every row count the pass kernel
is built for: logits, cosine similarities and the K/V rows it appends. This is what makes speculative output equal
autoregressive output on the GPU whatever the draft length (Section 1: verification keeps the full model's output)."""
import numpy as np
import pytest

import synth

pytestmark = pytest.mark.gpu

# widths that give a CTA several groups of weight rows, two activation windows at the larger row counts, grouped
# query attention, and a context that crosses a 128-key chunk border
SHAPES = [
    synth.DecoderShape(n_layers=3, d_model=512, n_heads=4, head_dim=128, d_ffn=1376, vocab=3001),
    synth.DecoderShape(n_layers=2, d_model=1024, n_heads=16, head_dim=64, d_ffn=2752, vocab=1777, n_kv_heads=4),
]


@pytest.mark.parametrize("shape", SHAPES, ids=["d512_hd128", "d1024_gqa"])
def test_every_row_count_is_bit_identical_to_one_row_passes(shape):
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=11, std=0.05)
    dec = asd.Decoder(shape, max_seq=200, max_draft=8)
    dec.load_weights_host(model)
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    prompt = synth.make_prompt(shape.vocab, 121, seed=12)          # rows 121.. cross the chunk border at 128
    cont = synth.make_prompt(shape.vocab, 16, seed=13)
    L = shape.n_layers

    def one_row_reference(n):
        dec.reset()
        t = dec.prefill(prompt)
        rows = [int(t)] + [int(v) for v in cont[:n - 1]]
        logits, cos, kv = [], [], []
        for r in rows:
            dec.decode_step(r)
            logits.append(dec.get_last_logits()[0].copy())
            ca, cm = dec.get_last_cosines()
            cos.append((ca[:, 0].copy(), cm[:, 0].copy()))
        for l in range(L):
            for p in range(len(prompt), len(prompt) + n):
                kv.append(dec.get_kv(l, p))
        return rows, logits, cos, kv

    rows9, logits1, cos1, _ = one_row_reference(9)
    for M in range(2, 10):
        dec.reset()
        dec.prefill(prompt)
        dec.verify(rows9[:M])
        lg = dec.get_last_logits()
        ca, cm = dec.get_last_cosines()
        assert lg.shape[0] == M
        for m in range(M):
            np.testing.assert_array_equal(lg[m], logits1[m], err_msg=f"logits, M={M}, row {m}")
            np.testing.assert_array_equal(ca[:, m], cos1[m][0], err_msg=f"attention cosines, M={M}, row {m}")
            np.testing.assert_array_equal(cm[:, m], cos1[m][1], err_msg=f"MLP cosines, M={M}, row {m}")
    # the K/V rows a 9-row pass appends are those of nine one-row passes (the verify above left them in the cache)
    kv_m = [dec.get_kv(l, p) for l in range(L) for p in range(len(prompt), len(prompt) + 9)]
    _, _, _, kv_1 = one_row_reference(9)
    for (a, b), (c, d) in zip(kv_m, kv_1):
        np.testing.assert_array_equal(a, c)
        np.testing.assert_array_equal(b, d)


def test_sixteen_row_prompt_passes_are_bit_identical_to_one_row_passes():
    import paper_2410_01028_b200 as asd
    shape = SHAPES[0]
    model = synth.make_model(shape, seed=21, std=0.05)
    dec = asd.Decoder(shape, max_seq=200, max_draft=8)
    dec.load_weights_host(model)
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    prompt = synth.make_prompt(shape.vocab, 16 * 8 + 16 + 7, seed=22)   # 9 passes of 16 rows, then 7 rows
    t1 = dec.prefill(prompt)
    l_rows = dec.get_last_logits()[-1].copy()
    ca_r, cm_r, n_r = dec.get_similarity()
    dec.reset()
    dec.prefill(prompt[:1])
    for t in prompt[1:]:
        t2 = dec.decode_step(int(t))
    np.testing.assert_array_equal(dec.get_last_logits()[0], l_rows)
    assert t1 == t2
    assert n_r == len(prompt)


@pytest.mark.parametrize("shape", SHAPES, ids=["d512_hd128", "d1024_gqa"])
def test_tagged_handoff_and_grid_barrier_variants_of_the_one_row_pass_agree_bit_for_bit(shape):
    """The one-row pass hands activations over as tagged words (no grid barrier); the debug flag makes it use the grid
    barrier like the multi-row passes. Same arithmetic, so logits, cosines and K/V must be identical."""
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=31, std=0.05)
    dec = asd.Decoder(shape, max_seq=300, max_draft=8)
    dec.load_weights_host(model)
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    prompt = synth.make_prompt(shape.vocab, 250, seed=32)           # decode steps cross the chunk border at 256
    cont = synth.make_prompt(shape.vocab, 10, seed=33)
    runs = []
    for barrier in (False, True):
        dec.reset()
        dec.set_debug(True, no_tagged_handoff=barrier)
        t = dec.prefill(prompt)
        logits, cos = [], []
        for r in [int(t)] + [int(v) for v in cont]:
            dec.decode_step(r)
            logits.append(dec.get_last_logits()[0].copy())
            ca, cm = dec.get_last_cosines()
            cos.append(np.concatenate([ca[:, 0], cm[:, 0]]))
        kv = [dec.get_kv(l, p) for l in range(shape.n_layers) for p in range(len(prompt), len(prompt) + 11)]
        runs.append((logits, cos, kv))
    dec.set_debug(True, no_tagged_handoff=False)
    for a, b in zip(runs[0][0], runs[1][0]):
        np.testing.assert_array_equal(a, b)
    for a, b in zip(runs[0][1], runs[1][1]):
        np.testing.assert_array_equal(a, b)
    for (ka, va), (kb, vb) in zip(runs[0][2], runs[1][2]):
        np.testing.assert_array_equal(ka, kb)
        np.testing.assert_array_equal(va, vb)
