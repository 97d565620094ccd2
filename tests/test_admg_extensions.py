"""The two opt-in extensions of the draft-model generator that the paper does not have: MLP sublayers removed by
their own similarity (the paper's Table 1 measures those similarities, Algorithm 1 never uses them), and C_l kept
running over the rows committed after the prompt with Algorithm 1 run again every few rounds.

CPU part: pins of the oracle (brute force over all masks; the running C_l against the definition of C_l applied to
prompt + emitted tokens; losslessness). GPU part: the library against the oracle.
"""
import itertools

import numpy as np
import pytest

import oracle
import synth
from helpers import COS_TOL, MASK_MARGIN

SMALL = synth.DecoderShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=50)
EXT = oracle.ADMG_ALL | oracle.USE_CS_MLP


@pytest.fixture(scope="module")
def small():
    return synth.make_model(SMALL, seed=7, std=0.2)


# ------------------------------------------------------------------ MLP threshold: brute force over all masks, L = 2
def _member_by_member(mask_attn, mask_mlp, Ca, Cm, alpha, alpha_mlp, m, n, flags):
    L = len(Ca)
    n_eff = n if flags & oracle.USE_RULE2 else 0
    for l in range(1, L + 1):
        guarded = l <= L - n_eff
        rule1 = bool(flags & oracle.USE_RULE1) and m >= 1 and any(l == j * m for j in range(1, L + 1)) and guarded
        cs_attn = bool(flags & oracle.USE_CS) and np.float32(Ca[l - 1]) >= np.float32(alpha) and guarded
        cs_mlp = bool(flags & oracle.USE_CS_MLP) and np.float32(Cm[l - 1]) >= np.float32(alpha_mlp) and guarded
        if bool(mask_attn[l - 1]) != (cs_attn or rule1) or bool(mask_mlp[l - 1]) != (cs_mlp or rule1):
            return False
    return True


@pytest.mark.parametrize("flags", [oracle.USE_CS_MLP, oracle.USE_CS | oracle.USE_CS_MLP, EXT,
                                   oracle.USE_CS_MLP | oracle.USE_RULE2])
def test_mlp_threshold_brute_force_two_layers(flags):
    alpha, alpha_mlp = 0.5, 0.7
    grid = [0.0, 0.5, 0.7, 0.9]
    masks = list(itertools.product((0, 1), repeat=2))
    for ca in itertools.product(grid, repeat=2):
        for cm in itertools.product(grid, repeat=2):
            Ca, Cm = np.array(ca, np.float32), np.array(cm, np.float32)
            for m in (1, 2):
                for n in (0, 1, 2):
                    got_a, got_m = oracle.admg_ext(Ca, Cm, alpha, alpha_mlp, m, n, flags)
                    sat = [(a, b) for a in masks for b in masks
                           if _member_by_member(a, b, Ca, Cm, alpha, alpha_mlp, m, n, flags)]
                    assert len(sat) == 1
                    assert sat[0] == (tuple(got_a.tolist()), tuple(got_m.tolist())), (ca, cm, m, n, flags)


def test_mlp_threshold_off_is_algorithm_1_and_attention_set_never_changes():
    rng = np.random.default_rng(5)
    for _ in range(200):
        L = int(rng.integers(1, 48))
        Ca = rng.uniform(0.5, 1.0, L).astype(np.float32)
        Cm = rng.uniform(0.5, 1.0, L).astype(np.float32)
        m, n = int(rng.integers(0, 6)), int(rng.integers(0, 6))
        for flags in range(8):
            ra, rm = oracle.admg(Ca, 0.9, m, n, flags)
            ea, em = oracle.admg_ext(Ca, Cm, 0.9, 0.8, m, n, flags)
            assert ea.tolist() == ra.tolist() and em.tolist() == rm.tolist()  # flag off: Algorithm 1 as printed
            xa, xm = oracle.admg_ext(Ca, Cm, 0.9, 0.8, m, n, flags | oracle.USE_CS_MLP)
            assert xa.tolist() == ra.tolist()      # the attention set is Algorithm 1's with or without the flag
            assert np.all(xm >= rm)                # the MLP set only grows
            n_eff = n if flags & oracle.USE_RULE2 else 0
            want = rm.astype(bool) | ((Cm >= np.float32(0.8)) & (np.arange(1, L + 1) <= L - n_eff))
            assert xm.astype(bool).tolist() == want.tolist()
    # inclusive comparison in float
    a = np.float32(0.8)
    Cm = np.array([a, np.nextafter(a, np.float32(0)), np.nextafter(a, np.float32(2))], np.float32)
    _, rm = oracle.admg_ext(np.zeros(3, np.float32), Cm, 2.0, float(a), 0, 0, oracle.USE_CS_MLP)
    assert rm.tolist() == [1, 0, 1]


# ------------------------------------------------------------------ running C_l
def _definition_of_c(model, tokens):
    """C_l as Section 3.2 defines it, over the given rows: one prefill of all of them."""
    o = oracle.Oracle(model, max_seq=len(tokens) + 1)
    o.prefill(tokens)
    return o.similarity()


@pytest.mark.parametrize("mode,k,refresh", [(oracle.MODE_AR, 0, 0), (oracle.MODE_SPEC, 3, 0), (oracle.MODE_SPEC, 4, 2),
                                            (oracle.MODE_SPEC, 2, 1)])
def test_running_similarity_is_the_mean_over_every_committed_row(small, mode, k, refresh):
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=21)
    o = oracle.Oracle(small, max_seq=64)
    ar, _, _ = o.generate(prompt, 20, mode=oracle.MODE_AR)
    ca0, cm0, n0 = o.similarity()
    assert n0 == 6  # off by default: the prompt rows only
    toks, _, st = o.generate(prompt, 20, mode=mode, draft_len=k, alpha=0.9, m=2, n=0,
                             flags=oracle.ADMG_ALL | oracle.RUNNING_C, refresh=refresh)
    assert toks.tolist() == ar.tolist()  # lossless whatever the masks did on the way
    ca, cm, n = o.similarity()
    # the committed rows are the prompt and every emitted token but the last
    assert n == 6 + 20 - 1
    da, dm, dn = _definition_of_c(small, np.concatenate([prompt, toks[:-1]]))
    assert dn == n
    np.testing.assert_allclose(ca, da, atol=2e-6)
    np.testing.assert_allclose(cm, dm, atol=2e-6)
    assert np.abs(ca - ca0).max() > 1e-4  # and it did move away from the prompt-only value


def test_refresh_installs_the_mask_of_the_refreshed_similarities(small):
    prompt = synth.make_prompt(SMALL.vocab, 6, seed=22)
    o = oracle.Oracle(small, max_seq=64)
    o.generate(prompt, 16, mode=oracle.MODE_SPEC, draft_len=3, alpha=0.9, alpha_mlp=0.9, m=0, n=0,
               flags=oracle.USE_CS | oracle.USE_CS_MLP | oracle.RUNNING_C, refresh=1)
    ca, cm, _ = o.similarity()
    # refresh = 1: the mask in force after the last round is Algorithm 1 on the final C_l
    want_a, want_m = oracle.admg_ext(ca, cm, 0.9, 0.9, 0, 0, oracle.USE_CS | oracle.USE_CS_MLP)
    got_a, got_m = o.admg_update(0.9, 0, 0, oracle.USE_CS | oracle.USE_CS_MLP, alpha_mlp=0.9)
    assert got_a.tolist() == want_a.tolist() and got_m.tolist() == want_m.tolist()


def test_single_steps_fold_their_committed_rows(small):
    prompt = synth.make_prompt(SMALL.vocab, 5, seed=23)
    o = oracle.Oracle(small, max_seq=32)
    ar, _, _ = o.generate(prompt, 8, mode=oracle.MODE_AR)
    o.reset()
    o.set_running_similarity(True)
    t1 = o.prefill(prompt)
    t2 = o.decode_step(t1)
    drafts = ar[2:5].copy()
    drafts[1] = (drafts[1] + 1) % SMALL.vocab  # second draft wrong: one accepted, two rows committed
    a, out = o.verify(np.concatenate([[t2], drafts]))
    assert a == 1
    ca, cm, n = o.similarity()
    assert n == 5 + 1 + 2
    da, dm, _ = _definition_of_c(small, np.concatenate([prompt, ar[:3]]))
    np.testing.assert_allclose(ca, da, atol=2e-6)
    np.testing.assert_allclose(cm, dm, atol=2e-6)
    o.set_running_similarity(False)


# ------------------------------------------------------------------ the library against the oracle
@pytest.mark.gpu
def test_gpu_mlp_threshold_equals_oracle():
    import paper_2410_01028_b200 as asd
    rng = np.random.default_rng(9)
    for _ in range(100):
        L = int(rng.integers(1, 48))
        Ca = rng.uniform(0.5, 1.0, L).astype(np.float32)
        Cm = rng.uniform(0.5, 1.0, L).astype(np.float32)
        m, n = int(rng.integers(0, 6)), int(rng.integers(0, 6))
        for flags in range(16):
            ga, gm = asd.admg_ext(Ca, Cm, 0.9, 0.8, m, n, flags)
            oa, om = oracle.admg_ext(Ca, Cm, 0.9, 0.8, m, n, flags)
            assert ga.tolist() == oa.tolist() and gm.tolist() == om.tolist()


@pytest.mark.gpu
def test_gpu_error_paths_of_the_extension_calls(tiny_model):
    import ctypes
    import paper_2410_01028_b200 as asd
    from paper_2410_01028_b200 import binding
    L = 4
    ca = np.full(L, 0.5, np.float32)
    ra, rm = np.zeros(L, np.uint8), np.zeros(L, np.uint8)
    p = binding.AdmgParams(0.9, 0, 0, asd.USE_CS_MLP, 0.9, 0)
    vp = lambda a: ctypes.c_void_p(a.ctypes.data)
    # the MLP threshold needs the MLP similarities
    assert asd.lib().asd_admg_ext(vp(ca), None, ctypes.c_int32(L), ctypes.byref(p), vp(ra), vp(rm)) == binding.ERR_ARG
    assert asd.lib().asd_admg(vp(ca), ctypes.c_int32(L), ctypes.byref(p), vp(ra), vp(rm)) == binding.ERR_ARG
    p.flags = asd.USE_CS  # without the flag they may be absent
    assert asd.lib().asd_admg_ext(vp(ca), None, ctypes.c_int32(L), ctypes.byref(p), vp(ra), vp(rm)) == 0
    assert asd.lib().asd_set_running_similarity(None, ctypes.c_int32(1)) == binding.ERR_ARG
    dec = asd.Decoder(synth.TINY, max_seq=64, max_draft=8)
    dec.load_weights_host(tiny_model)
    with pytest.raises(asd.AsdError):  # no pass has run the LM head yet
        dec.get_last_margins()
    dec.close()


@pytest.mark.gpu
@pytest.mark.parametrize("k,refresh", [(4, 0), (4, 2), (3, 1)])
def test_gpu_running_similarity_and_refreshed_masks(tiny_model, tiny_prompt, k, refresh):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    orc = oracle.Oracle(tiny_model, max_seq=128)
    flags = asd.USE_CS | asd.USE_RULE2 | asd.USE_CS_MLP | asd.RUNNING_C
    alpha, alpha_mlp = 0.9, 0.9
    ar, _ = dec.generate(tiny_prompt, 48, mode=asd.MODE_AR)
    sp, st = dec.generate(tiny_prompt, 48, mode=asd.MODE_SPEC, draft_len=k, alpha=alpha, alpha_mlp=alpha_mlp, m=0, n=1,
                          flags=flags, refresh=refresh)
    assert sp.tolist() == ar.tolist()  # speculative output equals autoregressive output bit for bit
    ca_g, cm_g, n_g = dec.get_similarity()
    assert n_g == 32 + 48 - 1
    # the oracle on the GPU's own token stream (the definition of C_l over the committed rows)
    orc.prefill(np.concatenate([tiny_prompt, sp[:-1]]))
    ca_o, cm_o, n_o = orc.similarity()
    assert n_o == n_g
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    # mask of the refreshed similarities: equal wherever the deciding margin is clear
    ga, gm = dec.admg_update(alpha, 0, 1, flags, alpha_mlp=alpha_mlp)
    oa, om = oracle.admg_ext(ca_o, cm_o, alpha, alpha_mlp, 0, 1, flags)
    clear_a, clear_m = np.abs(ca_o - alpha) > MASK_MARGIN, np.abs(cm_o - alpha_mlp) > MASK_MARGIN
    assert np.array_equal(ga[clear_a], oa[clear_a]) and np.array_equal(gm[clear_m], om[clear_m])
    # AR mode with the flag folds every decode step too
    _, _ = dec.generate(tiny_prompt, 48, mode=asd.MODE_AR, flags=asd.RUNNING_C)
    ca_a, cm_a, n_a = dec.get_similarity()
    assert n_a == n_g
    np.testing.assert_allclose(ca_a, ca_g, atol=1e-6)
    np.testing.assert_allclose(cm_a, cm_g, atol=1e-6)
    dec.close()


@pytest.mark.gpu
def test_gpu_single_steps_fold_their_committed_rows(tiny_model, tiny_prompt):
    import paper_2410_01028_b200 as asd
    dec = asd.Decoder(synth.TINY, max_seq=128, max_draft=8)
    dec.load_weights_host(tiny_model)
    ar, _ = dec.generate(tiny_prompt, 8, mode=asd.MODE_AR)
    dec.reset()
    dec.set_running_similarity(True)
    t1 = dec.prefill(tiny_prompt)
    t2 = dec.decode_step(t1)
    drafts = ar[2:5].copy()
    drafts[1] = (drafts[1] + 1) % synth.TINY.vocab
    a, _ = dec.verify(np.concatenate([[t2], drafts]))
    assert a == 1
    ca_g, cm_g, n = dec.get_similarity()
    assert n == 32 + 1 + 2
    orc = oracle.Oracle(tiny_model, max_seq=128)
    orc.prefill(np.concatenate([tiny_prompt, ar[:3]]))
    ca_o, cm_o, _ = orc.similarity()
    assert np.abs(ca_g - ca_o).max() <= COS_TOL and np.abs(cm_g - cm_o).max() <= COS_TOL
    dec.set_running_similarity(False)
    dec.close()
