"""Pins for the float64 oracle: nothing here compares the oracle with itself.

Each test fixes the oracle to something the mathematics determines: numerical
derivatives, invariants of softmax and of the normalisations, closed-form special
cases, a scalar triple-loop attention, equivalences between GQA and MHA, and an
independently formulated einsum version of the whole layer.
"""
import numpy as np
import pytest

from fbl_inputs import LayerConfig, get_config, make_inputs, scaled_config
from oracle import layer as orc
from oracle import naive


def tiny(norm="layernorm", causal=True, hq=4, hkv=2, residual=False, bias=True, B=2, T=7, D=12, hd=3, seed=11):
    return LayerConfig("tiny", B, T, D, hq, hkv, hd, "fp32", norm, causal, bias, residual, 1e-5, seed, 0.3)


def big_inputs(cfg):
    """Inputs with O(1) weights so every path carries signal (the 0.02 init hides sign errors)."""
    inp = make_inputs(cfg, affine_noise=True)
    return inp


VARIANTS = [
    dict(norm="layernorm", causal=True, hq=4, hkv=2),
    dict(norm="layernorm", causal=False, hq=2, hkv=2, residual=True),
    dict(norm="rmsnorm", causal=True, hq=4, hkv=1),
    dict(norm="rmsnorm", causal=False, hq=4, hkv=4, bias=False, residual=True),
]


def loss(cfg, inp):
    Y, _ = orc.layer_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                         inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    return float((Y * inp["dY"]).sum())


@pytest.mark.parametrize("kw", VARIANTS)
def test_finite_differences_every_gradient(kw):
    cfg = tiny(**kw)
    inp = big_inputs(cfg)
    _, _, g = orc.layer_fwd_bwd(cfg, inp)
    names = {"X": "dX", "Wq": "dWq", "Wk": "dWk", "Wv": "dWv", "Wo": "dWo", "gamma": "dgamma",
             "beta": "dbeta", "bq": "dbq", "bk": "dbk", "bv": "dbv", "bo": "dbo"}
    h = 1e-6
    for pname, gname in names.items():
        if inp[pname] is None:
            continue
        flat = inp[pname].reshape(-1)
        got = g[gname].reshape(-1)
        scale = np.abs(got).max() + 1e-3
        for i in range(flat.size):
            keep = flat[i]
            flat[i] = keep + h
            lp = loss(cfg, inp)
            flat[i] = keep - h
            lm = loss(cfg, inp)
            flat[i] = keep
            fd = (lp - lm) / (2 * h)
            assert abs(fd - got[i]) <= 2e-6 * scale + 2e-8, (pname, i, fd, got[i])


def test_finite_differences_config1_sampled():
    cfg = get_config(1)
    inp = make_inputs(cfg)
    _, _, g = orc.layer_fwd_bwd(cfg, inp)
    rng = np.random.default_rng(0)
    for pname, gname in [("X", "dX"), ("Wq", "dWq"), ("Wk", "dWk"), ("Wv", "dWv"), ("Wo", "dWo"),
                         ("gamma", "dgamma"), ("beta", "dbeta")]:
        flat, got = inp[pname].reshape(-1), g[gname].reshape(-1)
        scale = np.abs(got).max()
        for i in rng.choice(flat.size, 12, replace=False):
            keep = flat[i]
            flat[i] = keep + 1e-5
            lp = loss(cfg, inp)
            flat[i] = keep - 1e-5
            lm = loss(cfg, inp)
            flat[i] = keep
            assert abs((lp - lm) / 2e-5 - got[i]) <= 1e-6 * scale + 1e-9, (pname, i)


@pytest.mark.parametrize("causal", [True, False])
def test_softmax_rows_and_ds_rows(causal):
    rng = np.random.default_rng(1)
    T, hd = 9, 5
    q, k, v, dO = (rng.standard_normal((T, hd)) for _ in range(4))
    O, P, lse = orc.attention_head_fwd(q, k, v, 0.7, causal)
    assert np.allclose(P.sum(axis=1), 1.0, atol=1e-15)
    assert (P >= 0).all()
    if causal:
        assert (np.triu(P, 1) == 0).all()
        assert np.allclose(O[0], v[0], atol=1e-15)
    # LSE is the log of the un-normalised row sum
    S = 0.7 * q @ k.T
    mask = np.tril(np.ones((T, T), bool)) if causal else np.ones((T, T), bool)
    assert np.allclose(lse, np.log(np.where(mask, np.exp(S), 0).sum(1)), atol=1e-13)
    # D_i = sum_j P_ij dP_ij  ==  sum_d dO_id O_id, hence rows of dS sum to zero
    dP = dO @ v.T
    D1 = (P * dP).sum(1)
    D2 = (dO * O).sum(1)
    assert np.allclose(D1, D2, atol=1e-13)


def test_layer_ds_rows_sum_to_zero_via_dq():
    # with K rows all equal to one vector k0, dQ_i = scale * (sum_j dS_ij) k0 = 0
    cfg = tiny(bias=True)
    inp = big_inputs(cfg)
    inp["Wk"][:] = 0.0                      # K = bk for every token
    _, _, g = orc.layer_fwd_bwd(cfg, inp)
    assert np.abs(g["dQ"]).max() < 1e-14
    assert np.abs(g["dWq"]).max() < 1e-13


@pytest.mark.parametrize("causal", [True, False])
def test_against_triple_loop_attention(causal):
    rng = np.random.default_rng(2)
    q, k, v = (rng.standard_normal((6, 4)) for _ in range(3))
    O, P, _ = orc.attention_head_fwd(q, k, v, 0.5, causal)
    On, Pn = naive.naive_attention(q, k, v, 0.5, causal)
    assert np.allclose(O, On, atol=1e-14) and np.allclose(P, Pn, atol=1e-14)


@pytest.mark.parametrize("kw", VARIANTS)
def test_against_einsum_formulation(kw):
    cfg = tiny(**kw)
    inp = big_inputs(cfg)
    Y, _, g = orc.layer_fwd_bwd(cfg, inp)
    ref = naive.einsum_layer(cfg, inp)
    assert np.allclose(Y, ref["Y"], rtol=0, atol=1e-12 * np.abs(Y).max())
    for kname, val in ref.items():
        if kname == "Y" or (kname == "dbeta" and cfg.norm != "layernorm"):
            continue
        assert np.abs(g[kname] - val).max() <= 1e-12 * max(1.0, np.abs(val).max()), kname


def test_against_einsum_formulation_config1():
    cfg = get_config(1)
    inp = make_inputs(cfg)
    Y, _, g = orc.layer_fwd_bwd(cfg, inp)
    ref = naive.einsum_layer(cfg, inp)
    assert np.abs(Y - ref["Y"]).max() <= 1e-12 * np.abs(Y).max()
    for kname in ("dX", "dWq", "dWk", "dWv", "dWo", "dgamma", "dbeta"):
        assert np.abs(g[kname] - ref[kname]).max() <= 1e-12 * np.abs(ref[kname]).max(), kname


def test_dbk_is_zero():
    cfg = tiny()
    _, _, g = orc.layer_fwd_bwd(cfg, big_inputs(cfg))
    assert np.abs(g["dbk"]).max() < 1e-13 * np.abs(g["dbv"]).max()


@pytest.mark.parametrize("causal", [True, False])
def test_closed_form_uniform_attention(causal):
    cfg = tiny(causal=causal, hq=2, hkv=2, bias=False)
    inp = big_inputs(cfg)
    inp["Wq"][:] = 0.0
    Y, saved = orc.layer_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"])
    V = saved["V"]
    if causal:
        want = np.cumsum(V, axis=1) / np.arange(1, cfg.seq + 1)[None, :, None]
        lse = np.log(np.arange(1, cfg.seq + 1))
    else:
        want = np.broadcast_to(V.mean(axis=1, keepdims=True), V.shape)
        lse = np.full(cfg.seq, np.log(cfg.seq))
    assert np.allclose(saved["A"], want, atol=1e-14)
    assert np.allclose(saved["LSE"], lse[None, None, :], atol=1e-14)
    assert np.allclose(Y, want @ inp["Wo"], atol=1e-13)


def test_closed_form_single_token():
    cfg = tiny(T=1, B=3)
    inp = big_inputs(cfg)
    Y, _ = orc.layer_fwd(cfg, inp["X"], inp["gamma"], inp["beta"], inp["Wq"], inp["Wk"], inp["Wv"], inp["Wo"],
                         inp["bq"], inp["bk"], inp["bv"], inp["bo"])
    X = inp["X"]
    mu = X.mean(-1, keepdims=True)
    xn = (X - mu) / np.sqrt(X.var(-1, keepdims=True) + cfg.eps) * inp["gamma"] + inp["beta"]
    v = xn @ inp["Wv"] + inp["bv"]
    vrep = np.repeat(v.reshape(3, 1, cfg.n_kv_heads, cfg.head_dim), cfg.group, axis=2).reshape(3, 1, -1)
    assert np.allclose(Y, vrep @ inp["Wo"] + inp["bo"], atol=1e-13)


def test_norm_against_library_statistics():
    rng = np.random.default_rng(5)
    X = rng.standard_normal((3, 5, 16)) * 3 + 1
    gmm, bt = rng.standard_normal(16), rng.standard_normal(16)
    Xn, xhat, rstd, mu = orc.norm_fwd(X, gmm, bt, 1e-5, "layernorm")
    assert np.allclose(Xn, (X - np.mean(X, -1, keepdims=True)) / np.sqrt(np.var(X, -1, keepdims=True) + 1e-5) * gmm + bt)
    assert np.allclose(xhat.mean(-1), 0, atol=1e-14)
    Xr, xh, rs, _ = orc.norm_fwd(X, gmm, None, 0.0, "rmsnorm")
    assert np.allclose((xh ** 2).mean(-1), 1.0, atol=1e-13)
    assert np.allclose(Xr, X / np.linalg.norm(X, axis=-1, keepdims=True) * np.sqrt(16) * gmm)


def test_gqa_equals_mha_with_repeated_kv_blocks():
    cfg = tiny(hq=4, hkv=2, bias=True)
    inp = big_inputs(cfg)
    Y, _, g = orc.layer_fwd_bwd(cfg, inp)
    hd, G = cfg.head_dim, cfg.group
    rep = lambda W: np.concatenate([W[..., (h // G) * hd:(h // G + 1) * hd] for h in range(cfg.n_q_heads)], axis=-1)
    cfg_m = scaled_config(cfg, n_kv_heads=4)
    inp_m = dict(inp)
    for n in ("Wk", "Wv", "bk", "bv"):
        inp_m[n] = rep(inp[n])
    Ym, _, gm = orc.layer_fwd_bwd(cfg_m, inp_m)
    assert np.allclose(Y, Ym, atol=1e-13)
    assert np.allclose(g["dX"], gm["dX"], atol=1e-12)
    for n in ("dWk", "dWv", "dbk", "dbv"):
        full = gm[n]
        folded = np.concatenate([sum(full[..., (kv * G + r) * hd:(kv * G + r + 1) * hd] for r in range(G))
                                 for kv in range(cfg.n_kv_heads)], axis=-1)
        assert np.allclose(g[n], folded, atol=1e-12), n


def test_batch_structure():
    cfg = tiny(B=3)
    inp = big_inputs(cfg)
    Y, _, g = orc.layer_fwd_bwd(cfg, inp)
    acc = {}
    for b in range(3):
        one = dict(inp)
        one["X"], one["dY"] = inp["X"][b:b + 1], inp["dY"][b:b + 1]
        Yb, _, gb = orc.layer_fwd_bwd(scaled_config(cfg, batch=1), one)
        assert np.allclose(Y[b], Yb[0], atol=1e-13) and np.allclose(g["dX"][b], gb["dX"][0], atol=1e-13)
        for n in ("dWq", "dWk", "dWv", "dWo", "dgamma", "dbeta", "dbq", "dbv", "dbo"):
            acc[n] = acc.get(n, 0) + gb[n]
    for n, v in acc.items():
        assert np.allclose(g[n], v, atol=1e-12), n


def test_causality_and_permutation():
    cfg = tiny(causal=True)
    inp = big_inputs(cfg)
    t0 = 4
    Y, _, _ = orc.layer_fwd_bwd(cfg, inp)
    inp2 = {k: (None if v is None else v.copy()) for k, v in inp.items()}
    inp2["X"][:, t0:] += 1.0
    Y2, _, _ = orc.layer_fwd_bwd(cfg, inp2)
    assert np.array_equal(Y[:, :t0], Y2[:, :t0])
    inp3 = {k: (None if v is None else v.copy()) for k, v in inp.items()}
    inp3["dY"][:, t0:] = 0.0
    _, _, g3 = orc.layer_fwd_bwd(cfg, inp3)
    assert np.abs(g3["dX"][:, t0:]).max() == 0.0
    # non-causal: permuting tokens permutes Y and dX, leaves weight gradients unchanged
    cfgn = tiny(causal=False)
    perm = np.random.default_rng(3).permutation(cfgn.seq)
    Yn, _, gn = orc.layer_fwd_bwd(cfgn, inp)
    inpp = dict(inp)
    inpp["X"], inpp["dY"] = inp["X"][:, perm], inp["dY"][:, perm]
    Yp, _, gp = orc.layer_fwd_bwd(cfgn, inpp)
    assert np.allclose(Yp, Yn[:, perm], atol=1e-13) and np.allclose(gp["dX"], gn["dX"][:, perm], atol=1e-13)
    assert np.allclose(gp["dWk"], gn["dWk"], atol=1e-12)


def test_backward_is_linear_in_dy():
    cfg = tiny(residual=True)
    inp = big_inputs(cfg)
    _, _, g1 = orc.layer_fwd_bwd(cfg, inp)
    other = dict(inp)
    other["dY"] = np.random.default_rng(4).standard_normal(inp["dY"].shape)
    _, _, g2 = orc.layer_fwd_bwd(cfg, other)
    both = dict(inp)
    both["dY"] = 2.5 * inp["dY"] + other["dY"]
    _, _, g3 = orc.layer_fwd_bwd(cfg, both)
    for n in ("dX", "dWq", "dWk", "dWv", "dWo", "dgamma", "dbeta"):
        assert np.allclose(g3[n], 2.5 * g1[n] + g2[n], atol=1e-11), n


def test_norm_backward_invariants():
    cfg = tiny(norm="layernorm")
    inp = big_inputs(cfg)
    _, _, g = orc.layer_fwd_bwd(cfg, inp)
    assert np.abs(g["dX"].sum(-1)).max() < 1e-12          # shift invariance of LayerNorm
    cfg_r = tiny(norm="rmsnorm")
    inp_r = big_inputs(cfg_r)
    _, _, gr = orc.layer_fwd_bwd(scaled_config(cfg_r, eps=0.0), inp_r)
    assert np.abs((gr["dX"] * inp_r["X"]).sum(-1)).max() < 1e-11   # scale invariance (eps = 0)


def test_oracle_matches_its_committed_fixture():
    # Drift guard (not a pin to the paper): the oracle's values on two tiny seeded layers are stored under
    # tests/golden/ by a script that calls only oracle/; a change of the oracle's arithmetic changes them.
    import importlib.util
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_oracle_golden", os.path.join(here, "make_oracle_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = [ln.split() for ln in open(os.path.join(here, "oracle_layer_tiny.txt")) if not ln.startswith("#")]
    fresh = [ln.split() for ln in mod.lines()]
    assert len(stored) == len(fresh) == 14
    for s, f in zip(stored, fresh):
        assert s[:3] == f[:3]
        a, b = np.array(s[3:], dtype=np.float64), np.array(f[3:], dtype=np.float64)
        assert np.allclose(a, b, rtol=1e-12, atol=1e-14), (s[0], s[1])


def test_rope_is_a_position_dependent_rotation():
    # identity at position 0; norm-preserving; inverse undoes it; a textbook 2-D rotation for head_dim 2
    rng = np.random.default_rng(0)
    x = rng.normal(size=(2, 5, 12))
    y = orc.rope(x, 3, 10000.0)
    assert np.array_equal(y[:, 0], x[:, 0])
    assert np.abs(np.linalg.norm(y.reshape(2, 5, 3, 4), axis=-1) - np.linalg.norm(x.reshape(2, 5, 3, 4), axis=-1)).max() < 1e-12
    assert np.abs(orc.rope(y, 3, 10000.0, inverse=True) - x).max() < 1e-12
    z = orc.rope(np.array([[[1.0, 0.0], [1.0, 0.0], [0.0, 1.0]]]), 1, 10000.0)          # hd = 2: one pair, angle = t
    assert np.abs(z[0, 1] - [np.cos(1.0), np.sin(1.0)]).max() < 1e-15
    assert np.abs(z[0, 2] - [-np.sin(2.0), np.cos(2.0)]).max() < 1e-15
    # frequencies: pair i of an 8-wide head turns by t * base^(-2i/8)
    e = np.zeros((1, 4, 8)); e[0, :, 1] = 1.0
    w = orc.rope(e, 1, 100.0)
    assert np.abs(w[0, 3, 1] - np.cos(3 * 100.0 ** (-2 / 8))) < 1e-15 and np.abs(w[0, 3, 5] - np.sin(3 * 100.0 ** (-2 / 8))) < 1e-15


def test_rope_scores_depend_on_relative_position_only():
    # q_i . k_j after rotation depends on i - j: shifting every position by a constant leaves the scores unchanged
    rng = np.random.default_rng(1)
    q, k = rng.normal(size=(1, 6, 8)), rng.normal(size=(1, 6, 8))
    s0 = orc.rope(q, 2, 50.0).reshape(6, 2, 4).transpose(1, 0, 2) @ orc.rope(k, 2, 50.0).reshape(6, 2, 4).transpose(1, 2, 0)
    s7 = orc.rope(q, 2, 50.0, pos_offset=7).reshape(6, 2, 4).transpose(1, 0, 2) @ orc.rope(k, 2, 50.0, pos_offset=7).reshape(6, 2, 4).transpose(1, 2, 0)
    assert np.abs(s0 - s7).max() < 1e-12


@pytest.mark.parametrize("kw", [dict(norm="rmsnorm", causal=True, hq=4, hkv=2), dict(norm="layernorm", causal=False, hq=2, hkv=2, residual=True)])
def test_finite_differences_with_rope(kw):
    cfg = scaled_config(LayerConfig("tiny-rope", 2, 7, 12, kw["hq"], kw["hkv"], 4, "fp32", kw["norm"], kw["causal"], True,
                                    kw.get("residual", False), 1e-5, 13, 0.3), d_model=kw["hq"] * 4, rope_base=100.0)
    inp = big_inputs(cfg)
    _, _, g = orc.layer_fwd_bwd(cfg, inp)
    names = {"X": "dX", "Wq": "dWq", "Wk": "dWk", "Wv": "dWv", "Wo": "dWo", "gamma": "dgamma", "bq": "dbq", "bk": "dbk"}
    h = 1e-6
    for pname, gname in names.items():
        flat, got = inp[pname].reshape(-1), g[gname].reshape(-1)
        scale = np.abs(got).max() + 1e-3
        for i in range(0, flat.size, 3):
            keep = flat[i]
            flat[i] = keep + h
            lp = loss(cfg, inp)
            flat[i] = keep - h
            lm = loss(cfg, inp)
            flat[i] = keep
            assert abs((lp - lm) / (2 * h) - got[i]) <= 3e-6 * scale, (pname, i)
    # with the rotation in place the key bias no longer cancels: dbk is a real gradient now
    assert np.abs(g["dbk"]).max() > 1e-6
