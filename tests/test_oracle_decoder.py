"""Pins of the oracle's decoder, similarity accumulation and speculative loop.

Each test ties the oracle to something outside itself: a closed form, an
invariant of the mathematics, a special case that reduces to a numpy routine,
or the losslessness of greedy speculative decoding (Section 1).
"""
import dataclasses
import itertools
import math

import numpy as np
import pytest

import oracle
import synth

SMALL = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)
GQA = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50, n_kv_heads=2)


def f32(a):
    return synth.bf16_to_f32(a)


def bf(a):
    return synth.f32_to_bf16(np.asarray(a, np.float32))


@pytest.fixture(scope="module")
def small():
    return synth.make_model(SMALL, seed=7, std=0.2)  # larger std: activations of order 1 at d=64


# ------------------------------------------------------------------ fused sublayer product
def test_plain_matvec_equals_numpy_float64():
    W = synth.make_matrix_bf16((37, 72), seed=1, stream=1)
    x = synth.make_array_f32((3, 72), seed=1, stream=2)
    out, _ = oracle.fused_matvec(x, W, epilogue=0)
    ref = x.astype(np.float64) @ f32(W).astype(np.float64).T
    np.testing.assert_allclose(out, ref.astype(np.float32), rtol=0, atol=0)


def test_matvec_operand_orientation():
    # W[r][k] = 1 only at (r=2, k=5): out[m][2] = x[m][5], everything else 0  (catches a transposed operand)
    W = np.zeros((4, 8), np.float32)
    W[2, 5] = 1.0
    x = np.arange(16, dtype=np.float32).reshape(2, 8)
    out, _ = oracle.fused_matvec(x, bf(W), epilogue=0)
    want = np.zeros((2, 4), np.float32)
    want[:, 2] = x[:, 5]
    np.testing.assert_array_equal(out, want)


def test_rmsnorm_invariants():
    n = 64
    eye = bf(np.eye(n, dtype=np.float32))
    ones = bf(np.ones(n, np.float32))
    x = synth.make_array_f32((2, n), seed=2, stream=3, std=3.0)
    out, _ = oracle.fused_matvec(x, eye, epilogue=0, gain=ones, eps=0.0)
    # unit root-mean-square (up to the bf16 rounding of the normalised row, 2^-9 relative per element)
    np.testing.assert_allclose(np.sqrt((out.astype(np.float64) ** 2).mean(axis=1)), 1.0, atol=2e-3)
    # invariant to a positive rescaling of the input (power of two: exact)
    out4, _ = oracle.fused_matvec(4 * x, eye, epilogue=0, gain=ones, eps=0.0)
    np.testing.assert_array_equal(out, out4)
    # direction preserved
    for m in range(2):
        assert oracle.cosine(out[m], x[m]) > 0.99999
    # gain multiplies element-wise: gain 2 doubles (exact in bf16)
    out2, _ = oracle.fused_matvec(x, eye, epilogue=0, gain=bf(2 * np.ones(n, np.float32)), eps=0.0)
    np.testing.assert_array_equal(out2, 2 * out)
    # eps enters under the root: x = 0 gives 0, and a huge eps shrinks the output by 1/sqrt(eps)
    z, _ = oracle.fused_matvec(np.zeros((1, n), np.float32), eye, epilogue=0, gain=ones, eps=1e-5)
    assert not z.any()
    c = np.full((1, n), 1.0, np.float32)  # mean square 1; eps = 3 -> 1/sqrt(4) = 0.5
    h, _ = oracle.fused_matvec(c, eye, epilogue=0, gain=ones, eps=3.0)
    np.testing.assert_array_equal(h, np.full((1, n), 0.5, np.float32))


def test_swiglu_closed_forms():
    # one-hot rows make a = x_i and b = x_j exactly, so out = bf16(silu(x_i) * x_j)
    vals = np.array([[0.0, 1.0, -1.0, 20.0, -20.0, 0.5, -0.5, 2.0]], np.float32)
    eye = bf(np.eye(8, dtype=np.float32))
    ones_col = np.zeros((8, 8), np.float32)
    ones_col[:, 7] = 1.0  # b = x_7 = 2 for every output
    out, _ = oracle.fused_matvec(vals, eye, epilogue=1, W2=bf(ones_col))
    silu = out[0] / 2.0
    assert silu[0] == 0.0
    assert silu[1] == pytest.approx(1 / (1 + math.exp(-1)), rel=2 ** -8)
    assert silu[3] == pytest.approx(20.0, rel=2 ** -8)        # silu(x) -> x for large x
    assert abs(silu[4]) < 1e-7                                 # silu(x) -> 0 for very negative x
    # silu(x) - silu(-x) = x
    assert silu[1] - silu[2] == pytest.approx(1.0, abs=2 ** -7)
    assert silu[5] - silu[6] == pytest.approx(0.5, abs=2 ** -8)
    # the gate is the FIRST matrix: swapping the matrices changes the result
    out_sw, _ = oracle.fused_matvec(vals, bf(ones_col), epilogue=1, W2=eye)
    assert out_sw[0, 0] == 0.0 and out_sw[0, 1] == pytest.approx(2 / (1 + math.exp(-2)) * 1.0, rel=2 ** -8)


def test_residual_epilogue_orthogonal_update():
    # res = s*e_0, a = t*e_1  =>  cos = s/sqrt(s^2+t^2)
    W = np.zeros((4, 4), np.float32)
    W[1, 0] = 1.0
    x = np.array([[3.0, 0, 0, 0]], np.float32)
    res = np.array([[4.0, 0, 0, 0]], np.float32)
    out, cosv = oracle.fused_matvec(x, bf(W), epilogue=2, res=res)
    np.testing.assert_array_equal(out, np.array([[4.0, 3.0, 0, 0]], np.float32))
    assert cosv[0] == pytest.approx(0.8, abs=1e-7)


# ------------------------------------------------------------------ decoder special cases
def zero_out(model, **which):
    repl = {}
    for k, layers in which.items():
        a = getattr(model, k).copy()
        a[list(layers)] = 0
        repl[k] = a
    return dataclasses.replace(model, **repl)


def test_zero_output_projections_make_sublayers_the_identity(small):
    m = zero_out(small, wo=range(SMALL.n_layers), wd=range(SMALL.n_layers))
    o = oracle.Oracle(m, max_seq=16)
    toks = np.array([3, 11, 42, 7], np.int32)
    o.prefill(toks)
    last = o.last()
    assert np.all(last["cos_attn"] == 1.0) and np.all(last["cos_mlp"] == 1.0)
    ca, cm, n = o.similarity()
    assert n == 4 and np.all(ca == 1.0) and np.all(cm == 1.0)
    # the logits are then LM-head x RMSNorm(embedding row): a numpy product
    d = SMALL.d_model
    e = f32(m.embed)[toks].astype(np.float64)
    xn = e / np.sqrt((e ** 2).mean(axis=1, keepdims=True) + 1e-5) * f32(m.final_norm).astype(np.float64)
    xn = f32(bf(xn.astype(np.float32))).astype(np.float64)
    ref = xn @ f32(m.lm_head).astype(np.float64).T
    np.testing.assert_allclose(last["logits"], ref, rtol=1e-6, atol=1e-7)
    assert last["argmax"].tolist() == ref.argmax(axis=1).tolist()


def test_single_token_attention_returns_the_value_row(small):
    # S = 1: softmax over one key is 1, so the attention output is v itself and y = x + Wo v
    m1 = dataclasses.replace(small, shape=dataclasses.replace(SMALL, n_layers=1),
                             **{k: getattr(small, k)[:1] for k in
                                ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu", "wd")})
    m1 = zero_out(m1, wd=[0])
    o = oracle.Oracle(m1, max_seq=4)
    tok = 5
    o.prefill([tok])
    k, v = o.kv(0, 0)
    x = f32(m1.embed)[tok]
    xn, _ = oracle.fused_matvec(x[None], bf(np.eye(SMALL.d_model, dtype=np.float32)), gain=m1.attn_norm[0])
    v_ref, _ = oracle.fused_matvec(xn, m1.wv[0])
    np.testing.assert_array_equal(v, f32(bf(v_ref[0])))
    y, cosv = oracle.fused_matvec(v[None], m1.wo[0], epilogue=2, res=x[None])
    assert o.last()["cos_attn"][0, 0] == pytest.approx(float(cosv[0]), abs=1e-7)
    # rotary embedding at position 0 is the identity: k is the plain projection
    k_ref, _ = oracle.fused_matvec(xn, m1.wk[0])
    np.testing.assert_array_equal(k, f32(bf(k_ref[0])))


def test_zero_query_gives_uniform_causal_average(small):
    # Wq = 0 => all scores equal => the attention output at position p is the mean of v_0..v_p (keys 0..p inclusive)
    m1 = dataclasses.replace(small, shape=dataclasses.replace(SMALL, n_layers=1),
                             **{k: getattr(small, k)[:1] for k in
                                ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "wg", "wu", "wd")})
    m1 = zero_out(m1, wq=[0], wd=[0])
    # Wo = identity so that y - x exposes the attention output
    wo = bf(np.eye(SMALL.d_model, dtype=np.float32))[None]
    m1 = dataclasses.replace(m1, wo=wo)
    o = oracle.Oracle(m1, max_seq=8, flags=oracle.FLAG_NO_ROUNDING)
    toks = [1, 2, 3, 4, 5]
    # expose y through the cosine: instead read v rows and compare cos(x, x + mean v)
    o.prefill(toks)
    got = o.last()["cos_attn"][0]
    vs = np.stack([o.kv(0, p)[1] for p in range(len(toks))]).astype(np.float64)
    for p, t in enumerate(toks):
        x = f32(m1.embed)[t].astype(np.float64)
        y = x + vs[: p + 1].mean(axis=0)
        ref = float(x @ y / (np.linalg.norm(x) * np.linalg.norm(y)))
        assert got[p] == pytest.approx(ref, abs=2e-6)


def test_rotary_embedding_angle_pairing_and_direction(small):
    # Layer 1 sees position-independent inputs (the embedding row), so feeding the same token at every
    # position makes the cached key at position p the rotation by p*theta_j of the same vector.
    o = oracle.Oracle(small, max_seq=16, flags=oracle.FLAG_NO_ROUNDING)
    o.prefill([9] * 12)
    hd, half = SMALL.head_dim, SMALL.head_dim // 2
    ks = np.stack([o.kv(0, p)[0] for p in range(12)]).astype(np.float64).reshape(12, SMALL.n_heads, hd)
    a, b = ks[..., :half], ks[..., half:]          # element j is paired with j + hd/2
    np.testing.assert_allclose(a ** 2 + b ** 2, (a ** 2 + b ** 2)[:1].repeat(12, 0), rtol=1e-5)  # a rotation
    ang = np.arctan2(b, a)
    theta = 10000.0 ** (-2.0 * np.arange(half) / hd)
    for p in range(1, 12):
        delta = np.angle(np.exp(1j * (ang[p] - ang[0] - p * theta)))  # wrap to (-pi, pi]
        np.testing.assert_allclose(delta, 0.0, atol=1e-5)


def test_prefill_equals_sequential_decode(small):
    toks = synth.make_prompt(SMALL.vocab, 9, seed=3)
    a = oracle.Oracle(small, max_seq=16)
    t1 = a.prefill(toks)
    la = a.last()
    b = oracle.Oracle(small, max_seq=16)
    b.prefill(toks[:1])
    for t in toks[1:]:
        out = b.decode_step(int(t))
    lb = b.last()
    assert out == t1
    np.testing.assert_array_equal(la["logits"][-1], lb["logits"][0])
    for l in range(SMALL.n_layers):
        for p in range(9):
            np.testing.assert_array_equal(a.kv(l, p)[0], b.kv(l, p)[0])
            np.testing.assert_array_equal(a.kv(l, p)[1], b.kv(l, p)[1])


def test_chunked_prefill_equals_one_shot_and_acs_is_a_mean(small):
    toks = synth.make_prompt(SMALL.vocab, 10, seed=4)
    a = oracle.Oracle(small, max_seq=16)
    a.prefill(toks)
    per_row = a.last()
    ca, cm, n = a.similarity()
    assert n == 10
    np.testing.assert_allclose(ca, per_row["cos_attn"].astype(np.float64).mean(axis=1), atol=1e-7)
    np.testing.assert_allclose(cm, per_row["cos_mlp"].astype(np.float64).mean(axis=1), atol=1e-7)
    b = oracle.Oracle(small, max_seq=16)
    b.prefill(toks[:3]); b.prefill(toks[3:4]); t1 = b.prefill(toks[4:])
    cb, cmb, nb = b.similarity()
    assert nb == 10 and t1 == per_row["argmax"][-1]
    np.testing.assert_array_equal(ca, cb)
    np.testing.assert_array_equal(cm, cmb)
    # S = 1: C is that row's cosine
    c = oracle.Oracle(small, max_seq=16)
    c.prefill(toks[:1])
    c1, _, _ = c.similarity()
    np.testing.assert_array_equal(c1, c.last()["cos_attn"][:, 0])


def test_head_and_ffn_permutation_invariance(small):
    rng = np.random.default_rng(0)
    hp = rng.permutation(SMALL.n_heads)
    idx = (hp[:, None] * SMALL.head_dim + np.arange(SMALL.head_dim)[None]).ravel()
    fp = rng.permutation(SMALL.d_ffn)
    perm = dataclasses.replace(
        small, wq=small.wq[:, idx], wk=small.wk[:, idx], wv=small.wv[:, idx], wo=small.wo[:, :, idx],
        wg=small.wg[:, fp], wu=small.wu[:, fp], wd=small.wd[:, :, fp])
    perm = dataclasses.replace(perm, **{k: np.ascontiguousarray(getattr(perm, k)) for k in
                                         ("wq", "wk", "wv", "wo", "wg", "wu", "wd")})
    toks = synth.make_prompt(SMALL.vocab, 6, seed=5)
    a = oracle.Oracle(small, max_seq=8); a.prefill(toks)
    b = oracle.Oracle(perm, max_seq=8); b.prefill(toks)
    np.testing.assert_allclose(a.last()["logits"], b.last()["logits"], rtol=0, atol=2e-2 * np.abs(a.last()["logits"]).max() * 0.05)
    np.testing.assert_allclose(a.last()["cos_attn"], b.last()["cos_attn"], atol=1e-4)


def test_grouped_query_attention_equals_replicated_heads():
    g = synth.make_model(GQA, seed=11, std=0.2)
    hd = GQA.head_dim
    rep = np.repeat(np.arange(GQA.kv_heads), GQA.n_heads // GQA.kv_heads)
    idx = (rep[:, None] * hd + np.arange(hd)[None]).ravel()
    mha_shape = dataclasses.replace(GQA, n_kv_heads=0)
    mha = dataclasses.replace(g, shape=mha_shape, wk=np.ascontiguousarray(g.wk[:, idx]),
                              wv=np.ascontiguousarray(g.wv[:, idx]))
    toks = synth.make_prompt(GQA.vocab, 7, seed=6)
    a = oracle.Oracle(g, max_seq=8); a.prefill(toks)
    b = oracle.Oracle(mha, max_seq=8); b.prefill(toks)
    np.testing.assert_array_equal(a.last()["logits"], b.last()["logits"])


def _numpy_decoder(model, toks):
    """Matrix-form float64 decoder without any intermediate rounding (an independent restatement)."""
    s = model.shape
    W = lambda a: f32(a).astype(np.float64)
    h = W(model.embed)[toks]
    S = len(toks)
    hd, half = s.head_dim, s.head_dim // 2
    pos = np.arange(S)[:, None]
    theta = 10000.0 ** (-2.0 * np.arange(half) / hd)
    cs, sn = np.cos(pos * theta), np.sin(pos * theta)

    def norm(x, g):
        return x / np.sqrt((x ** 2).mean(axis=1, keepdims=True) + 1e-5) * W(g)

    def rope(x, nh):
        x = x.reshape(S, nh, hd)
        a, b = x[..., :half], x[..., half:]
        return np.concatenate([a * cs[:, None] - b * sn[:, None], b * cs[:, None] + a * sn[:, None]], axis=-1)

    coss = []
    for l in range(s.n_layers):
        xn = norm(h, model.attn_norm[l])
        q = rope(xn @ W(model.wq[l]).T, s.n_heads)
        k = rope(xn @ W(model.wk[l]).T, s.kv_heads)
        v = (xn @ W(model.wv[l]).T).reshape(S, s.kv_heads, hd)
        grp = s.n_heads // s.kv_heads
        out = np.zeros((S, s.n_heads, hd))
        for hh in range(s.n_heads):
            sc = q[:, hh] @ k[:, hh // grp].T / math.sqrt(hd)
            sc = np.where(np.tril(np.ones((S, S), bool)), sc, -np.inf)
            p = np.exp(sc - sc.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            out[:, hh] = p @ v[:, hh // grp]
        y = h + out.reshape(S, -1) @ W(model.wo[l]).T
        ca = (h * y).sum(1) / np.linalg.norm(h, axis=1) / np.linalg.norm(y, axis=1)
        yn = norm(y, model.mlp_norm[l])
        g_, u_ = yn @ W(model.wg[l]).T, yn @ W(model.wu[l]).T
        z = y + (g_ / (1 + np.exp(-g_)) * u_) @ W(model.wd[l]).T
        cm = (y * z).sum(1) / np.linalg.norm(y, axis=1) / np.linalg.norm(z, axis=1)
        coss.append((ca, cm))
        h = z
    return norm(h, model.final_norm) @ W(model.lm_head).T, coss


@pytest.mark.parametrize("shape,seed", [(SMALL, 7), (GQA, 11)])
def test_unrounded_oracle_equals_matrix_form_float64(shape, seed):
    model = synth.make_model(shape, seed=seed, std=0.2)
    toks = synth.make_prompt(shape.vocab, 8, seed=8)
    o = oracle.Oracle(model, max_seq=8, flags=oracle.FLAG_NO_ROUNDING)
    o.prefill(toks)
    last = o.last()
    ref, coss = _numpy_decoder(model, toks)
    np.testing.assert_allclose(last["logits"], ref, rtol=0, atol=1e-4 * np.abs(ref).max())
    for l, (ca, cm) in enumerate(coss):
        np.testing.assert_allclose(last["cos_attn"][l], ca, atol=1e-5)
        np.testing.assert_allclose(last["cos_mlp"][l], cm, atol=1e-5)


def test_bf16_rounding_points_stay_within_the_logit_tolerance(tiny_model, tiny_prompt):
    a = oracle.Oracle(tiny_model, max_seq=32); a.prefill(tiny_prompt)
    b = oracle.Oracle(tiny_model, max_seq=32, flags=oracle.FLAG_NO_ROUNDING); b.prefill(tiny_prompt)
    la, lb = a.last(), b.last()
    tol = 2e-2 * np.abs(lb["logits"]).max(axis=1, keepdims=True)
    assert np.all(np.abs(la["logits"] - lb["logits"]) <= tol)
    assert np.abs(la["cos_attn"] - lb["cos_attn"]).max() < 1e-3
    assert np.abs(la["cos_mlp"] - lb["cos_mlp"]).max() < 1e-3


# ------------------------------------------------------------------ draft model and speculative loop
def test_empty_mask_draft_equals_full_model_and_everything_is_accepted(small):
    o = oracle.Oracle(small, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=9)
    o.set_skip_mask([0, 0], [0, 0])
    toks, _, st = o.generate(prompt, 20, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=4)
    assert st["accepted"] == st["drafted"] > 0
    ar, _, _ = o.generate(prompt, 20, mode=oracle.MODE_AR)
    assert toks.tolist() == ar.tolist()


def test_removed_sublayers_with_zero_projection_are_always_accepted(small):
    m = zero_out(small, wo=[0], wd=[1])
    o = oracle.Oracle(m, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=10)
    o.set_skip_mask([1, 0], [0, 1])
    toks, _, st = o.generate(prompt, 24, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=5)
    assert st["accepted"] == st["drafted"] > 0
    ar, _, _ = o.generate(prompt, 24, mode=oracle.MODE_AR)
    assert toks.tolist() == ar.tolist()


def test_speculative_output_is_lossless_for_every_mask_and_draft_length(small):
    o = oracle.Oracle(small, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 5, seed=12)
    max_new = 18
    ar, _, st_ar = o.generate(prompt, max_new, mode=oracle.MODE_AR)
    assert st_ar["full_passes"] == max_new - 1
    for bits in itertools.product((0, 1), repeat=4):
        for k in range(0, 9):
            o.set_skip_mask(bits[:2], bits[2:])
            toks, _, st = o.generate(prompt, max_new, mode=oracle.MODE_SPEC_MANUAL_MASK, draft_len=k)
            assert toks.tolist() == ar.tolist(), (bits, k)
            assert 0 <= st["accepted"] <= st["drafted"]
            # every round emits between 1 and k+1 tokens; committed = prompt + emitted - 1
            assert st["rounds"] <= max_new - 1 and (max_new - 1) <= st["rounds"] * (k + 1)
            assert max_new - 1 == st["accepted"] + st["rounds"]
            assert o.positions()[0] == len(prompt) + max_new - 1


def test_verify_accepts_the_longest_matching_prefix(small):
    o = oracle.Oracle(small, max_seq=64)
    prompt = synth.make_prompt(SMALL.vocab, 5, seed=13)
    ar, _, _ = o.generate(prompt, 8, mode=oracle.MODE_AR)
    for n_good in range(0, 5):
        o.reset()
        t1 = o.prefill(prompt)
        assert t1 == ar[0]
        drafts = ar[1:5].copy()
        if n_good < 4:
            drafts[n_good] = (drafts[n_good] + 1) % SMALL.vocab  # first wrong draft
        a, out = o.verify(np.concatenate([[t1], drafts]))
        assert a == n_good
        assert out.tolist() == ar[1:n_good + 2].tolist()  # accepted drafts, then M's own token
        assert o.positions() == (len(prompt) + n_good + 1, len(prompt) + n_good + 1)
        # decoding continues correctly from the committed state
        assert o.decode_step(int(out[-1])) == ar[n_good + 2]


def test_admg_generate_on_tiny_config(tiny_model, tiny_prompt):
    o = oracle.Oracle(tiny_model, max_seq=128)
    ar, margins, _ = o.generate(tiny_prompt, 64, mode=oracle.MODE_AR)
    ca, _, n = o.similarity()
    assert n == 32 and np.all(ca <= 1.0) and np.all(ca >= -1.0)
    for (m, n_) in [(3, 2), (2, 1)]:
        sp, margins2, st = o.generate(tiny_prompt, 64, mode=oracle.MODE_SPEC, draft_len=4, m=m, n=n_)
        assert sp.tolist() == ar.tolist()
        np.testing.assert_array_equal(margins, margins2)
        skip_a, skip_m = o.admg_update(0.985, m, n_)
        ra, rm = oracle.admg(ca, 0.985, m, n_)
        assert skip_a.tolist() == ra.tolist() and skip_m.tolist() == rm.tolist()


def test_error_codes(small):
    o = oracle.Oracle(small, max_seq=4)
    with pytest.raises(oracle.OracleError) as e:
        o.prefill([1, 2, 3, 4, 5])
    assert e.value.code == oracle.ERR_OVERFLOW
    with pytest.raises(oracle.OracleError) as e:
        o.prefill([SMALL.vocab])
    assert e.value.code == oracle.ERR_ARG
    with pytest.raises(oracle.OracleError) as e:
        o.similarity()
    assert e.value.code == oracle.ERR_STATE


# ------------------------------------------------------------------ the bf16 roundings inside a sublayer (R5, R7)
# Both cases are built from one-hot embeddings (RMSNorm turns e_i into exactly 8 e_i at d = 64: 1/sqrt(1/64 + 1e-5)
# = 7.9974, whose nearest bf16 value is 8) and a read-out row e_0 - e_1 in the output projection, so that the
# sublayer's output is the DIFFERENCE of two intermediate values that agree after the rounding and differ by 0.25
# before it. With the rounding the sublayer adds exactly nothing and its cosine is exactly 1; without it the
# residual moves by 0.25 e_0 and the cosine is 1/sqrt(1 + 0.25^2).
ONE_LAYER = synth.DecoderShape(n_layers=1, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)


def _blank_one_layer_model():
    s = ONE_LAYER
    d, f, V = s.d_model, s.d_ffn, s.vocab
    z = lambda *shape: np.zeros(shape, np.float32)
    embed, lm = z(V, d), z(V, d)
    embed[0, 0] = embed[1, 1] = 1.0          # token 0 -> e_0, token 1 -> e_1
    lm[0, 0] = lm[1, 1] = 1.0                # logit 0 reads element 0 of the final normalised state, logit 1 element 1
    ones = np.ones(d, np.float32)
    return dict(embed=embed, lm_head=lm, final_norm=ones, attn_norm=ones[None].copy(), wq=z(1, d, d), wk=z(1, d, d),
                wv=z(1, d, d), wo=z(1, d, d), mlp_norm=ones[None].copy(), wg=z(1, f, d), wu=z(1, f, d), wd=z(1, d, f))


def _as_model(parts):
    return synth.SynthModel(shape=ONE_LAYER, seed=0, **{k: bf(v) for k, v in parts.items()})


def test_attention_output_is_rounded_to_bf16_before_the_output_projection():
    # Wq = 0: uniform attention. Position 1 (token 1 after token 0) averages v_0 and v_1:
    #   element 0: (256 + 1.5) / 2 = 128.75 -> bf16 129 (spacing 1 between 128 and 256);  element 1: (129 + 129) / 2 = 129
    # W_o row 0 = e_0 - e_1: o_0 = 129 - 129 = 0 with the rounding R5, 128.75 - 129 = -0.25 without it.
    p = _blank_one_layer_model()
    p["wv"][0, 0, 0], p["wv"][0, 0, 1] = 32.0, 0.1875          # v[0] = 8 * 32 = 256 for token 0, 8 * 0.1875 = 1.5 for token 1
    p["wv"][0, 1, 0] = p["wv"][0, 1, 1] = 16.125               # v[1] = 129 for both tokens
    p["wo"][0, 0, 0], p["wo"][0, 0, 1] = 1.0, -1.0
    o = oracle.Oracle(_as_model(p), max_seq=4)
    o.prefill([0, 1])
    np.testing.assert_array_equal(o.kv(0, 0)[1][:2], [256.0, 129.0])
    np.testing.assert_array_equal(o.kv(0, 1)[1][:2], [1.5, 129.0])
    last = o.last()
    # position 0 attends to itself only: o_0 = 256 - 129 = 127 on top of x = e_0 -> y = 128 e_0, still parallel to x
    assert last["cos_attn"][0, 0] == 1.0
    # position 1: the rounded average makes o vanish, y = x = e_1 exactly
    assert last["cos_attn"][0, 1] == 1.0
    assert last["logits"][1, 0] == 0.0 and last["logits"][1, 1] == 8.0
    # the same case without any bf16 rounding: y = e_1 - 0.25 e_0 (up to the un-rounded norm factor 7.9974 / 8)
    u = oracle.Oracle(_as_model(p), max_seq=4, flags=oracle.FLAG_NO_ROUNDING)
    u.prefill([0, 1])
    assert u.last()["cos_attn"][0, 1] == pytest.approx(1 / math.sqrt(1 + 0.25 ** 2), abs=1e-4)
    assert u.last()["logits"][1, 0] < -1.0


def test_swiglu_product_is_rounded_to_bf16_before_the_down_projection():
    # attention is the identity (W_o = 0); the MLP sees yn = 8 e_1 for token 1.
    #   t_0 = silu(20) * 8.0625 = 161.25 -> bf16 161;  t_1 = silu(23) * 7 = 161   (silu(g) = g to float precision for g >= 20)
    # W_d row 0 = e_0 - e_1: dn_0 = 161 - 161 = 0 with the rounding R7, 0.25 without it.
    p = _blank_one_layer_model()
    p["wg"][0, 0, 1], p["wu"][0, 0, 1] = 2.5, 1.0078125        # g_0 = 20, u_0 = 8.0625
    p["wg"][0, 1, 1], p["wu"][0, 1, 1] = 2.875, 0.875          # g_1 = 23, u_1 = 7
    p["wd"][0, 0, 0], p["wd"][0, 0, 1] = 1.0, -1.0
    o = oracle.Oracle(_as_model(p), max_seq=4)
    o.prefill([1])
    last = o.last()
    assert last["cos_attn"][0, 0] == 1.0
    assert last["cos_mlp"][0, 0] == 1.0                         # z = y exactly
    assert last["logits"][0, 0] == 0.0 and last["logits"][0, 1] == 8.0
    u = oracle.Oracle(_as_model(p), max_seq=4, flags=oracle.FLAG_NO_ROUNDING)
    u.prefill([1])
    assert u.last()["cos_mlp"][0, 0] == pytest.approx(1 / math.sqrt(1 + 0.25 ** 2), abs=1e-4)
    assert u.last()["logits"][0, 0] > 1.0
