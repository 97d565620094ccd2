"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C ABI."""
import dataclasses

import numpy as np
import pytest

import oracle
import synth
from helpers import (COS_TOL, MARGIN, MASK_MARGIN, argmax_rows_agree, assert_cos_close, assert_logits_close,
                     teacher_forced_compare, verify_outcomes_agree)

pytestmark = pytest.mark.gpu

SMALL = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)
GQA = synth.DecoderShape(n_layers=3, d_model=128, n_heads=8, head_dim=16, d_ffn=200, vocab=77, n_kv_heads=2)
MID = synth.DecoderShape(n_layers=6, d_model=512, n_heads=4, head_dim=128, d_ffn=1376, vocab=3001)


def make_pair(shape, max_seq, seed=0, std=0.02, max_draft=8):
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=seed, std=std)
    dec = asd.Decoder(shape, max_seq=max_seq, max_draft=max_draft)
    dec.load_weights_host(model)
    orc = oracle.Oracle(model, max_seq=max_seq)
    return model, dec, orc


@pytest.fixture(scope="module")
def tiny_pair(tiny_model):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    return dec, oracle.Oracle(tiny_model, max_seq=128)


# ------------------------------------------------------------------ config 1: the tiny decoder end to end
def test_tiny_prefill_similarity_logits_and_kv(tiny_pair, tiny_prompt):
    dec, orc = tiny_pair
    dec.reset(); orc.reset()
    dec.set_debug(True)
    t_g, t_o = dec.prefill(tiny_prompt), orc.prefill(tiny_prompt)
    last = orc.last()
    ca_g, cm_g, n_g = dec.get_similarity()
    ca_o, cm_o, n_o = orc.similarity()
    assert n_g == n_o == 32
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    # the last prefill pass holds the last rows of the prompt
    ca, cm = dec.get_last_cosines()
    rows = ca.shape[1]
    assert_cos_close(ca, last["cos_attn"][:, -rows:])
    assert_cos_close(cm, last["cos_mlp"][:, -rows:])
    assert_logits_close(dec.get_last_logits(), last["logits"][-rows:])
    # token ids of those rows (the last one is t_1), wherever the oracle's top-2 gap decides them
    assert argmax_rows_agree(dec.get_last_logits(), last, slice(-rows, None)) >= rows // 2
    assert t_g == int(np.argmax(dec.get_last_logits()[-1]))
    # K/V cache, bf16. Layer 0 depends on the embedding, one RMSNorm and one product only: nearly every element is
    # identical, the rest are one-ulp rounding flips. Deeper layers inherit flips: one flipped element of K, V or of the
    # attention output moves the hidden state of every later row that attends to it by up to ~1e-3 of its scale and
    # flips many roundings there, so below layer 0 the bound is one ulp of the value plus 1e-2 of the row's scale.
    for l in range(synth.TINY.n_layers):
        flips = total = 0
        for p in (0, 1, 7, 8, 31):
            kg, vg = dec.get_kv(l, p)
            ko, vo = orc.kv(l, p)
            for g, o in ((synth.bf16_to_f32(kg), ko), (synth.bf16_to_f32(vg), vo)):
                assert np.all(np.abs(g - o) <= 2 ** -7 * np.abs(o) + (0.0 if l == 0 else 1e-2) * np.abs(o).max())
                flips += int((g != o).sum()); total += g.size
        if l == 0:
            assert flips <= 0.01 * total


def test_tiny_teacher_forced_decode(tiny_pair, tiny_prompt):
    dec, orc = tiny_pair
    res = teacher_forced_compare(dec, orc, tiny_prompt, 64)
    assert res.soft <= 8 and res.decided >= 32


def test_tiny_generate_ar_spec_bit_exact_and_matches_oracle(tiny_pair, tiny_prompt):
    import paper_2410_01028_b200 as asd
    dec, orc = tiny_pair
    ref, margins, _ = orc.generate(tiny_prompt, 64)
    ar, st_ar = dec.generate(tiny_prompt, 64, mode=asd.MODE_AR)
    assert st_ar["full_passes"] == 63
    # up to the first low-margin step the GPU must reproduce the oracle's tokens
    first_soft = next((i for i in range(64) if margins[i] <= MARGIN), 64)
    assert first_soft >= 4 and ar[:first_soft].tolist() == ref[:first_soft].tolist()
    for (m, n) in [(3, 2), (2, 1), (1, 0)]:
        for k in (1, 4, 8):
            sp, st = dec.generate(tiny_prompt, 64, mode=asd.MODE_SPEC, draft_len=k, m=m, n=n)
            assert sp.tolist() == ar.tolist(), (m, n, k)   # lossless, bit exact on the GPU
            assert st["accepted"] + st["rounds"] == 63
            assert dec.positions()[0] == 32 + 63
    # paper defaults remove nothing at L=4 (rule 1 needs l <= L-n = 2): the draft is the full model
    sp, st = dec.generate(tiny_prompt, 64, mode=asd.MODE_SPEC, draft_len=4, m=3, n=2)
    if np.all(np.abs(orc.similarity()[0][:2] - 0.985) > MASK_MARGIN) and np.all(orc.similarity()[0][:2] < 0.985):
        assert st["accepted"] == st["drafted"]


def test_tiny_skip_masks_match_oracle(tiny_pair, tiny_prompt):
    import paper_2410_01028_b200 as asd
    dec, orc = tiny_pair
    dec.reset(); orc.reset()
    dec.prefill(tiny_prompt); orc.prefill(tiny_prompt)
    C = orc.similarity()[0]
    for alpha in (0.985, 0.7, 0.6):
        for (m, n, flags) in [(3, 2, 7), (2, 1, 7), (2, 1, asd.USE_CS), (2, 1, asd.USE_CS | asd.USE_RULE2),
                              (2, 1, asd.USE_RULE1 | asd.USE_RULE2)]:
            ga, gm = dec.admg_update(alpha, m, n, flags)
            oa, om = orc.admg_update(alpha, m, n, flags)
            assert gm.tolist() == om.tolist()
            decided = np.abs(C - alpha) > MASK_MARGIN
            assert np.array_equal(ga[decided], oa[decided])


def test_tiny_draft_and_verify_calls_match_oracle(tiny_pair, tiny_prompt):
    dec, orc = tiny_pair
    decided_drafts = decided_verifies = 0
    for mask in ([0, 1, 0, 0], [0, 0, 1, 0]), ([1, 1, 1, 1], [1, 1, 1, 1]), ([0, 0, 0, 0], [0, 0, 0, 0]):
        dec.reset(); orc.reset()
        t = orc.prefill(tiny_prompt)
        dec.prefill(tiny_prompt)
        dec.set_skip_mask(*mask); orc.set_skip_mask(*mask)
        for _ in range(3):
            row_o, row_g = [t], [t]
            for j in range(4):
                row_o.append(orc.draft_step(row_o[-1]))
                m_o = orc.last()["margin"][0]
                row_g.append(dec.draft_step(row_g[-1]))
                ca, cm = dec.get_last_cosines()
                if row_g[:-1] == row_o[:-1]:
                    assert_cos_close(ca, orc.last()["cos_attn"])
                    assert_cos_close(cm, orc.last()["cos_mlp"])
                    if m_o > MARGIN:
                        assert row_g[-1] == row_o[-1]
                        decided_drafts += 1
            assert dec.positions() == orc.positions()
            a_o, out_o = orc.verify(row_o)
            margins = orc.last()["margin"]
            a_g, out_g = dec.verify(row_o)          # same drafted row into both
            decided_verifies += verify_outcomes_agree(a_g, out_g, a_o, out_o, margins)
            assert dec.positions()[0] == dec.positions()[1]
            if (a_g, out_g.tolist()) != (a_o, out_o.tolist()):
                break
            t = int(out_o[-1])
    assert decided_drafts >= 12 and decided_verifies >= 3     # the comparisons above did decide tokens


# ------------------------------------------------------------------ other shapes: odd sizes, GQA, several tiles
@pytest.mark.parametrize("shape,std,S,new", [(SMALL, 0.2, 5, 12), (GQA, 0.1, 19, 10), (MID, 0.02, 300, 24)])
def test_other_shapes_teacher_forced(shape, std, S, new):
    _, dec, orc = make_pair(shape, max_seq=S + new + 16, seed=3, std=std)
    prompt = synth.make_prompt(shape.vocab, S, seed=2)
    teacher_forced_compare(dec, orc, prompt, new)
    ca_g, cm_g, _ = dec.get_similarity()
    ca_o, cm_o, _ = orc.similarity()
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL


def test_mid_spec_equals_ar_for_every_draft_length_and_masks():
    import paper_2410_01028_b200 as asd
    _, dec, orc = make_pair(MID, max_seq=400, seed=3)
    prompt = synth.make_prompt(MID.vocab, 250, seed=4)   # 250 -> positions cross the 256-key chunk boundary
    ar, _ = dec.generate(prompt, 40, mode=asd.MODE_AR)
    rng = np.random.default_rng(0)
    for k in range(0, 9):
        mask = (rng.integers(0, 2, MID.n_layers), rng.integers(0, 2, MID.n_layers))
        dec.set_skip_mask(*mask)
        sp, st = dec.generate(prompt, 40, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=k)
        assert sp.tolist() == ar.tolist(), k
        assert st["accepted"] + st["rounds"] == 39
    dec.set_skip_mask(np.zeros(MID.n_layers), np.zeros(MID.n_layers))
    sp, st = dec.generate(prompt, 40, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=5)
    assert sp.tolist() == ar.tolist() and st["accepted"] == st["drafted"]   # empty mask: every draft accepted
    # a second run is bit-identical (no order-dependent reductions)
    sp2, _ = dec.generate(prompt, 40, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=5)
    assert sp2.tolist() == sp.tolist()


def test_prefill_equals_sequential_decode_on_gpu():
    _, dec, _ = make_pair(SMALL, max_seq=64, seed=3, std=0.2)
    prompt = synth.make_prompt(SMALL.vocab, 21, seed=5)
    dec.set_debug(True)
    t1 = dec.prefill(prompt)
    l1 = dec.get_last_logits()[-1]
    kv1 = [dec.get_kv(l, p) for l in range(2) for p in range(21)]
    dec.reset()
    dec.prefill(prompt[:1])
    for t in prompt[1:]:
        t2 = dec.decode_step(int(t))
    l2 = dec.get_last_logits()[0]
    kv2 = [dec.get_kv(l, p) for l in range(2) for p in range(21)]
    assert t1 == t2
    np.testing.assert_array_equal(l1, l2)      # row m of an M-row pass is bit-identical to a 1-row pass
    for (a, b), (c, d) in zip(kv1, kv2):
        np.testing.assert_array_equal(a, c); np.testing.assert_array_equal(b, d)


def test_zero_output_projection_gives_cosine_one_and_full_acceptance():
    import paper_2410_01028_b200 as asd
    model = synth.make_model(SMALL, seed=7, std=0.2)
    wo, wd = model.wo.copy(), model.wd.copy()
    wo[0] = 0; wd[1] = 0
    model = dataclasses.replace(model, wo=wo, wd=wd)
    dec = asd.Decoder(SMALL, max_seq=64)
    dec.load_weights_host(model)
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=10)
    dec.prefill(prompt)
    ca, cm = dec.get_last_cosines()
    assert np.all(ca[0] == 1.0) and np.all(cm[1] == 1.0)
    dec.set_skip_mask([1, 0], [0, 1])
    sp, st = dec.generate(prompt, 24, mode=asd.MODE_SPEC_MANUAL_MASK, draft_len=5)
    ar, _ = dec.generate(prompt, 24, mode=asd.MODE_AR)
    assert sp.tolist() == ar.tolist() and st["accepted"] == st["drafted"] > 0


# ------------------------------------------------------------------ the fused sublayer kernel on its own
def _run_fused(M, n_in, n_rows, epi, norm, seed):
    import torch
    import paper_2410_01028_b200 as asd
    dev = torch.device("cuda:0")
    W = synth.make_matrix_bf16((n_rows, n_in), seed=seed, stream=1)
    gain = synth.make_matrix_bf16((n_in,), seed=seed, stream=2, std=0.02, mean=1.0) if norm else None
    if norm:
        x = synth.make_array_f32((M, n_in), seed=seed, stream=3, std=1.5)
        x_dev = torch.from_numpy(x).to(dev)
    else:
        x = synth.make_array_f32((M, n_in), seed=seed, stream=3, std=1.0)      # bf16-representable
        x_dev = torch.from_numpy(synth.f32_to_bf16(x).view(np.int16)).to(dev).view(torch.bfloat16)
    W_dev = torch.from_numpy(W.view(np.int16)).to(dev).view(torch.bfloat16)
    g_dev = torch.from_numpy(gain.view(np.int16)).to(dev).view(torch.bfloat16) if norm else None
    scratch = torch.zeros(asd.fused_gemv_scratch_bytes(), dtype=torch.uint8, device=dev)
    cos_dev = torch.zeros(16, dtype=torch.float32, device=dev)
    res = None
    if epi == asd.EPI_PLAIN:
        out = torch.empty((M, n_rows), dtype=torch.float32, device=dev)
        W_o, W2_o = W, None
    elif epi == asd.EPI_SWIGLU:
        out = torch.empty((M, n_rows // 2), dtype=torch.bfloat16, device=dev)
        W_o, W2_o = np.ascontiguousarray(W[0::2]), np.ascontiguousarray(W[1::2])
    else:
        res = synth.make_array_f32((M, n_rows), seed=seed, stream=4, std=1.0)
        out = torch.from_numpy(res.copy()).to(dev)
        W_o, W2_o = W, None
    for _ in range(2):   # twice: the scratch counter must come back to zero
        if epi == asd.EPI_RESIDUAL:
            out.copy_(torch.from_numpy(res))
        asd.fused_gemv(x_dev, W_dev, epi, out, gain=g_dev, cos=cos_dev, scratch=scratch)
        torch.cuda.synchronize()
    ref, ref_cos = oracle.fused_matvec(x, W_o, epilogue=epi, gain=gain, W2=W2_o, res=res)
    got = out.float().cpu().numpy()
    return got, ref, cos_dev.cpu().numpy()[:M], ref_cos


@pytest.mark.parametrize("M", [1, 2, 5, 9])
@pytest.mark.parametrize("n_in,n_rows", [(256, 688 * 2), (688, 256), (1032, 51), (2048, 2048), (2048, 5504)])
def test_fused_gemv_against_oracle(M, n_in, n_rows):
    import paper_2410_01028_b200 as asd
    for epi, norm in [(asd.EPI_PLAIN, True), (asd.EPI_PLAIN, False), (asd.EPI_RESIDUAL, False), (asd.EPI_RESIDUAL, True),
                      (asd.EPI_SWIGLU, True)]:
        if epi == asd.EPI_SWIGLU and n_rows % 2:
            continue
        got, ref, cos_g, cos_o = _run_fused(M, n_in, n_rows, epi, norm, seed=n_in + n_rows + M)
        scale = np.abs(ref).max()
        if epi == asd.EPI_SWIGLU:
            # bf16 outputs: one-ulp flips allowed
            assert np.all(np.abs(got - ref) <= 2 ** -7 * np.abs(ref) + 1e-3 * scale)
        elif norm:
            # the normalised input is rounded to bf16 on both sides; a rounding flip moves one product by 2^-8
            assert np.all(np.abs(got - ref) <= 2e-3 * scale)
        else:
            assert np.all(np.abs(got - ref) <= 1e-5 * scale)
        if epi == asd.EPI_RESIDUAL:
            assert np.abs(cos_g - cos_o).max() <= (COS_TOL if norm else 1e-5)


def test_error_paths_on_the_host():
    import paper_2410_01028_b200 as asd
    model, dec, _ = make_pair(SMALL, max_seq=8, seed=1, std=0.2)
    with pytest.raises(asd.AsdError) as e:
        dec.prefill(np.arange(9) % SMALL.vocab)
    assert e.value.code == -4                       # overflow of max_seq
    with pytest.raises(asd.AsdError) as e:
        dec.prefill([SMALL.vocab])
    assert e.value.code == -1                       # token out of range
    with pytest.raises(asd.AsdError) as e:
        dec.get_similarity()
    assert e.value.code == -2                       # nothing prefetched yet
    dec.prefill([1, 2, 3, 4, 5, 6])
    with pytest.raises(asd.AsdError) as e:
        dec.verify([1, 2, 3, 4])                    # 6 + 4 > 8
    assert e.value.code == -4
    a, out = dec.verify([1, 2])                     # 6 + 2 <= 8 still fine
    assert 0 <= a <= 1
    fresh = asd.Decoder(SMALL, max_seq=8)
    with pytest.raises(asd.AsdError) as e:
        fresh.prefill([1])
    assert e.value.code == -2                       # weights not loaded
    # the context survives every one of these errors
    dec.reset()
    assert isinstance(dec.prefill([1, 2, 3]), int)


def test_weights_from_file_equal_weights_from_host(tmp_path):
    import paper_2410_01028_b200 as asd
    model, dec, _ = make_pair(SMALL, max_seq=32, seed=1, std=0.2)
    path = tmp_path / "w.bin"
    with open(path, "wb") as fh:
        for k in ("embed", "lm_head", "final_norm", "attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu", "wd"):
            fh.write(np.ascontiguousarray(getattr(model, k)).tobytes())
    dec2 = asd.Decoder(SMALL, max_seq=32)
    dec2.load_weights_file(str(path))
    prompt = synth.make_prompt(SMALL.vocab, 7, seed=1)
    assert dec.generate(prompt, 12)[0].tolist() == dec2.generate(prompt, 12)[0].tolist()
    with open(path, "ab") as fh:
        fh.truncate(100)
    with pytest.raises(asd.AsdError) as e:
        dec2.load_weights_file(str(path))
    assert e.value.code == -7


def test_bounded_device_wait_runs_out_and_the_context_recovers(tiny_model, tiny_prompt):
    """Every spin of the pass kernel has a cycle budget. Here the barrier in front of the last stage is told to wait
    for one arrival that never comes, with the budget cut to about a millisecond: the pass must still end, the call
    must report ASD_ERR_DEVICE_TIMEOUT with where it gave up, and after asd_reset the same context decodes as before."""
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    want, _ = dec.generate(tiny_prompt, 24, mode=asd.MODE_AR)
    dec.reset()
    t = dec.prefill(tiny_prompt)
    dec.set_debug(record_logits=False, short_waits=True)              # a short budget alone changes nothing
    t2 = dec.decode_step(t)
    assert t2 == want[1]
    dec.set_debug(record_logits=False, short_waits=True, missing_arrival=True)
    with pytest.raises(asd.AsdError) as e:
        dec.decode_step(t2)
    assert e.value.code == asd.binding.ERR_DEVICE_TIMEOUT
    assert "grid barrier" in str(e.value) and "stage" in str(e.value)
    with pytest.raises(asd.AsdError) as e:                           # the error is sticky until the context is reset
        dec.set_debug(record_logits=False)
        dec.decode_step(t2)
    assert e.value.code == asd.binding.ERR_DEVICE_TIMEOUT
    dec.reset()
    got, _ = dec.generate(tiny_prompt, 24, mode=asd.MODE_AR)
    assert got.tolist() == want.tolist()
    sp, _ = dec.generate(tiny_prompt, 24, mode=asd.MODE_SPEC, draft_len=4, m=2, n=1)
    assert sp.tolist() == want.tolist()
