"""GPU parity of the dense prompt path (tcgen05 GEMMs + causal flash attention + row kernels) through the C ABI:
the GEMM building block against the oracle's matrix product, and prompts processed in ASD_PREFILL_GEMM mode
against the CPU oracle (similarities, first token, logits, K/V cache) and against ASD_PREFILL_ROWS."""
import numpy as np
import pytest

import oracle
import synth
from helpers import COS_TOL, MARGIN, argmax_rows_agree, assert_cos_close, assert_logits_close, teacher_forced_compare

pytestmark = pytest.mark.gpu

MID = synth.DecoderShape(n_layers=6, d_model=512, n_heads=4, head_dim=128, d_ffn=1376, vocab=3001)
GQA64 = synth.DecoderShape(n_layers=3, d_model=512, n_heads=8, head_dim=64, d_ffn=520, vocab=501, n_kv_heads=2)


def _pair(shape, max_seq, seed=0, std=0.02):
    import paper_2410_01028_b200 as asd
    model = synth.make_model(shape, seed=seed, std=std)
    dec = asd.Decoder(shape, max_seq=max_seq, max_draft=8)
    dec.load_weights_host(model)
    return model, dec, oracle.Oracle(model, max_seq=max_seq)


# ------------------------------------------------------------------ the GEMM on its own
# fp32 accumulation of K products against the oracle's double accumulation: the error of one output is at most
# K * 2^-24 of the sum of the magnitudes of its products, which for these zero-mean inputs is below
# 1e-5 of the largest output for K <= 1032 (measured: 1.5e-6).
@pytest.mark.parametrize("M,N,K", [(1, 32, 64), (128, 128, 64), (37, 200, 72), (130, 256, 256), (300, 1376, 256),
                                   (257, 256, 688), (200, 768, 1032), (600, 4608, 512)])
def test_gemm_bf16_against_oracle(M, N, K):
    import torch
    import paper_2410_01028_b200 as asd
    dev = torch.device("cuda:0")
    A = synth.make_matrix_bf16((M, K), seed=M + N + K, stream=1, std=1.0)
    W = synth.make_matrix_bf16((N, K), seed=M + N + K, stream=2, std=0.05)
    A_d = torch.from_numpy(A.view(np.int16)).to(dev).view(torch.bfloat16)
    W_d = torch.from_numpy(W.view(np.int16)).to(dev).view(torch.bfloat16)
    C = torch.full((M, N), float("nan"), dtype=torch.float32, device=dev)
    status = torch.ones(8, dtype=torch.int32, device=dev)
    for _ in range(2):
        asd.gemm_bf16(A_d, W_d, C, status)
    torch.cuda.synchronize()
    assert status.tolist() == [0] * 8
    ref, _ = oracle.fused_matvec(synth.bf16_to_f32(A), W, epilogue=0)
    got = C.cpu().numpy()
    assert np.all(np.abs(got - ref) <= 1e-5 * np.abs(ref).max())


def test_gemm_bf16_rejects_bad_arguments():
    import torch
    import paper_2410_01028_b200 as asd
    dev = torch.device("cuda:0")
    A = torch.zeros((4, 60), dtype=torch.bfloat16, device=dev)   # K not a multiple of 8
    W = torch.zeros((8, 60), dtype=torch.bfloat16, device=dev)
    C = torch.zeros((4, 8), dtype=torch.float32, device=dev)
    st = torch.zeros(8, dtype=torch.int32, device=dev)
    with pytest.raises(asd.AsdError):
        asd.gemm_bf16(A, W, C, st)


# ------------------------------------------------------------------ prompts through the dense path
def _kv_close(dec, orc, layers, positions):
    """bf16 K/V rows against the oracle's. Layer 0 depends on the embedding, one RMSNorm and one product only: nearly
    every element is identical and the rest are one-ulp rounding flips. Deeper layers inherit those flips: one
    flipped element of K, V or of the attention output (2^-8 of its value) moves the hidden state of every later
    row that attends to it by up to ~1e-3 of its scale, which in turn flips many roundings there; so the bound is
    one ulp of the value plus 1e-2 of the row's scale (measured worst case 5.3e-3 four layers deep)."""
    for l in range(layers):
        flips = total = 0
        for p in positions:
            kg, vg = dec.get_kv(l, p)
            ko, vo = orc.kv(l, p)
            for g, o in ((synth.bf16_to_f32(kg), ko), (synth.bf16_to_f32(vg), vo)):
                assert np.all(np.abs(g - o) <= 2 ** -7 * np.abs(o) + (0.0 if l == 0 else 1e-2) * np.abs(o).max())
                flips += int((g != o).sum()); total += g.size
        if l == 0:
            assert flips <= 0.01 * total


def test_tiny_prompt_through_the_dense_path_matches_oracle(tiny_model, tiny_prompt):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    orc = oracle.Oracle(tiny_model, max_seq=128)
    dec.set_debug(True)
    dec.set_prefill_mode(asd.PREFILL_GEMM)
    t_g, t_o = dec.prefill(tiny_prompt), orc.prefill(tiny_prompt)
    last = orc.last()
    decided = argmax_rows_agree(dec.get_last_logits(), last, slice(-1, None))
    assert t_g == int(np.argmax(dec.get_last_logits()[-1]))
    ca_g, cm_g, n_g = dec.get_similarity()
    ca_o, cm_o, n_o = orc.similarity()
    assert n_g == n_o == 32
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    # the last prompt row: cosines from the dense path, logits from the LM-head stage of the pass kernel on its hidden state
    ca, cm = dec.get_last_cosines()
    assert ca.shape[1] == 1
    assert_cos_close(ca, last["cos_attn"][:, -1:])
    assert_cos_close(cm, last["cos_mlp"][:, -1:])
    assert_logits_close(dec.get_last_logits(), last["logits"][-1:])
    _kv_close(dec, orc, synth.TINY.n_layers, (0, 1, 7, 8, 30, 31))
    # and decoding continues from that cache exactly as the oracle does
    assert dec.positions() == (32, 32)
    t = t_o
    for _ in range(8):
        o = orc.decode_step(t)
        g = dec.decode_step(t)
        decided += argmax_rows_agree(dec.get_last_logits(), orc.last())
        assert g == int(np.argmax(dec.get_last_logits()[0]))
        assert_logits_close(dec.get_last_logits(), orc.last()["logits"])
        t = o
    assert decided >= 4                                       # tokens were compared, not only logits


@pytest.mark.parametrize("shape,std,S", [(MID, 0.02, 300), (GQA64, 0.05, 203)])
def test_dense_path_matches_oracle_and_row_passes(shape, std, S):
    import paper_2410_01028_b200 as asd
    _, dec, orc = _pair(shape, max_seq=S + 40, seed=3, std=std)
    prompt = synth.make_prompt(shape.vocab, S, seed=2)
    dec.set_prefill_mode(asd.PREFILL_GEMM)
    res = teacher_forced_compare(dec, orc, prompt, 12)       # prefill, then 11 teacher-forced steps on its cache
    assert res.soft <= 3 and res.decided >= 6
    ca_g, cm_g, n_g = dec.get_similarity()
    ca_o, cm_o, n_o = orc.similarity()
    assert n_g == n_o == S
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    _kv_close(dec, orc, shape.n_layers, (0, 63, 64, 127, 128, S - 2, S - 1))
    # both prompt paths of the library agree to rounding
    dec.reset()
    dec.set_prefill_mode(asd.PREFILL_ROWS)
    dec.prefill(prompt)
    ca_r, cm_r, _ = dec.get_similarity()
    assert np.abs(ca_g - ca_r).max() <= COS_TOL and np.abs(cm_g - cm_r).max() <= COS_TOL


def test_dense_path_in_several_chunks_and_appended_prompts():
    """A prompt longer than one chunk of the dense path (2048 rows), then a second prompt appended to the same
    context: positions, similarities and the cache follow the oracle."""
    import paper_2410_01028_b200 as asd
    shape = synth.DecoderShape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ffn=344, vocab=301)
    S1, S2 = 2100, 70
    _, dec, orc = _pair(shape, max_seq=S1 + S2 + 20, seed=5, std=0.05)
    p1 = synth.make_prompt(shape.vocab, S1, seed=7)
    p2 = synth.make_prompt(shape.vocab, S2, seed=8)
    dec.set_debug(True)
    t_g, t_o = dec.prefill(p1), orc.prefill(p1)              # default mode: dense path, chunks of 2048 + 51 rows, then 1 row
    assert orc.last()["margin"][-1] > MARGIN and t_g == t_o  # (this seed's first token is decided by a clear gap)
    assert_logits_close(dec.get_last_logits(), orc.last()["logits"][-1:])
    t_g, t_o = dec.prefill(p2), orc.prefill(p2)              # appended at position 2100: 69 dense rows + 1
    assert orc.last()["margin"][-1] > MARGIN and t_g == t_o
    assert_logits_close(dec.get_last_logits(), orc.last()["logits"][-1:])
    assert dec.positions() == (S1 + S2, S1 + S2)
    ca_g, cm_g, n_g = dec.get_similarity()
    ca_o, cm_o, n_o = orc.similarity()
    assert n_g == n_o == S1 + S2
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    _kv_close(dec, orc, shape.n_layers, (0, 2047, 2048, 2098, 2099, 2100, S1 + S2 - 1))
    assert dec.get_stats()["prefill_rows"] == S1 + S2


def test_dense_path_refused_where_the_shape_does_not_allow_it():
    import paper_2410_01028_b200 as asd
    small = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)
    _, dec, _ = _pair(small, max_seq=64, seed=3, std=0.2)
    with pytest.raises(asd.AsdError) as e:
        dec.set_prefill_mode(asd.PREFILL_GEMM)
    assert e.value.code == asd.binding.ERR_ARG
    assert isinstance(dec.prefill(np.arange(40) % small.vocab), int)   # default mode falls back to the row passes
