"""Pins for the decoder half of the CPU checker (Algorithm 2, Sec. 3.1, Sec. 4.1, Appendix
"Inference Detail").

The dense layer is pinned to a composition of textbook torch-CPU operators; the rotary
step to its complex-number form and its relative-position property; the cached step to the
identities that hold for any correct implementation of per-token K/V reuse.
"""
import math

import numpy as np
import pytest
import torch

from oracle import vla_cache_oracle as orc
from paper_2502_02175_b200 import synth


def _tiny(seed=0, n_layers=2):
    cfg = synth.tiny_config().with_layers(n_layers)
    model = synth.make_model(cfg, seed)
    ids = synth.make_prompt_ids(cfg, seed)[0]
    rng = np.random.default_rng(seed + 1)
    feats = synth.f32_to_bf16(rng.standard_normal((cfg.n_vision, cfg.hidden), dtype=np.float32))
    return cfg, model, ids, feats


def _t(bits):
    """bf16 bit patterns -> fp64 torch tensor through torch's own bfloat16 type (not the checker's widening)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).double()


def test_widen_bf16_matches_torch_bfloat16():
    """The checker's bit widening against torch.bfloat16 on every class of pattern: normals of both signs,
    subnormals, zeros, infinities, and (as a set) NaNs."""
    rng = np.random.default_rng(0)
    bits = rng.integers(0, 1 << 16, size=20000, dtype=np.uint16)
    special = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x3F80, 0xBF80,
                        0x7FC0, 0xFFC1], dtype=np.uint16)
    bits = np.concatenate([bits, special])
    with np.errstate(invalid="ignore"):          # widening a signalling NaN raises the flag
        got = orc.widen_bf16(bits)
    want = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))
    assert got[len(bits) - len(special) + 2] == 2.0 ** -133 and np.isposinf(got[len(bits) - len(special) + 8])
    # the memoised form is the same conversion
    orc.WIDEN_CACHE_MAX = 2
    try:
        with np.errstate(invalid="ignore"):
            assert np.array_equal(orc._widen_cached(bits)[~nan], want[~nan])
            assert np.array_equal(orc._widen_cached(bits)[~nan], want[~nan])
    finally:
        orc.WIDEN_CACHE_MAX = 0
        orc._widen_cache.clear()


def _torch_rope(x, cos, sin):
    """x [L, H, d]; positions 0..L-1; rotate-half convention."""
    half = x.shape[-1] // 2
    c = torch.cat([cos, cos], dim=-1)[:, None, :]
    s = torch.cat([sin, sin], dim=-1)[:, None, :]
    rot = torch.cat([-x[..., half:], x[..., :half]], dim=-1)
    return x * c + rot * s


def _torch_layer(cfg, lw, h, cos, sin, mask=None, rb=lambda t: t):
    """Textbook Llama layer over a full sequence in fp64: causal, or with a boolean mask [L, L].  ``rb`` is applied to
    every operand of a matrix product other than the weights (identity, or a rounding to bf16 by torch)."""
    L, H, d = h.shape[0], cfg.n_heads, cfg.head_dim
    F = torch.nn.functional
    xn = rb(F.rms_norm(h, (cfg.hidden,), _t(lw["g_attn"]), cfg.rms_eps))
    q = rb(_torch_rope(F.linear(xn, _t(lw["wq"])).view(L, H, d), cos, sin))
    k = rb(_torch_rope(F.linear(xn, _t(lw["wk"])).view(L, H, d), cos, sin))
    v = rb(F.linear(xn, _t(lw["wv"])).view(L, H, d))
    if mask is None and rb(torch.tensor([1.0 + 2.0 ** -12], dtype=torch.float64)).item() != 1.0:
        o = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1), is_causal=True)
    elif mask is not None:
        o = F.scaled_dot_product_attention(q.transpose(0, 1), k.transpose(0, 1), v.transpose(0, 1), attn_mask=mask)
    else:       # rounded probabilities: the softmax has to be written out
        sc = torch.einsum("qhd,khd->hqk", q, k) / math.sqrt(d)
        sc = sc.masked_fill(~torch.tril(torch.ones(L, L, dtype=torch.bool)), float("-inf"))
        o = torch.einsum("hqk,khd->hqd", rb(torch.softmax(sc, dim=-1)), v)
    h = h + F.linear(rb(o.transpose(0, 1).reshape(L, H * d)), _t(lw["wo"]))
    xn = rb(F.rms_norm(h, (cfg.hidden,), _t(lw["g_mlp"]), cfg.rms_eps))
    return h + F.linear(rb(F.silu(F.linear(xn, _t(lw["w_gate"]))) * F.linear(xn, _t(lw["w_up"]))), _t(lw["w_down"])), k, v


def test_full_prefill_equals_textbook_layer():
    cfg, model, ids, feats = _tiny()
    L = cfg.seq_len
    h0 = orc.input_rows(cfg, model, feats, ids)
    cos = torch.from_numpy(model["rope_cos"][:L].astype(np.float64))
    sin = torch.from_numpy(model["rope_sin"][:L].astype(np.float64))
    ht = torch.from_numpy(h0[:L].copy())
    cache = orc.new_cache(cfg)
    hidden = h0.copy()
    for l in range(cfg.n_layers):
        orc.layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden, np.arange(L),
                          model["rope_cos"], model["rope_sin"])
        ht, k, v = _torch_layer(cfg, model["layers"][l], ht, cos, sin)
        np.testing.assert_allclose(cache.K[l][:L], k.numpy(), atol=1e-10)
        np.testing.assert_allclose(cache.V[l][:L], v.numpy(), atol=1e-10)
        np.testing.assert_allclose(hidden[:L], ht.numpy(), atol=1e-10)


def test_input_rows_layout():
    cfg, model, ids, feats = _tiny()
    h = orc.input_rows(cfg, model, feats, ids)
    emb = orc.widen_bf16(model["embed"])
    np.testing.assert_array_equal(h[0], emb[ids[0]])
    np.testing.assert_array_equal(h[cfg.n_text_pre + cfg.n_vision], emb[ids[cfg.n_text_pre]])
    np.testing.assert_array_equal(h[cfg.seq_len - 1], emb[ids[-1]])
    want = torch.nn.functional.linear(_t(feats), _t(model["proj"])).numpy()
    np.testing.assert_allclose(h[cfg.n_text_pre:cfg.n_text_pre + cfg.n_vision], want, atol=1e-12)
    assert np.all(h[cfg.seq_len:] == 0)


def test_input_rows_of_the_recomputed_positions_only():
    """Projecting only the vision rows layer 0 recomputes: those rows equal the full projection, every other vision row
    stays zero, and a whole cached step gives the same bits either way (a row skipped in layer 0 is skipped everywhere)."""
    cfg, model, ids, feats = _tiny(5)
    v0, v1 = cfg.n_text_pre, cfg.n_text_pre + cfg.n_vision
    rows0 = np.asarray([0, v0 + 3, v0 + 4, v0 + 40, v1, v1 + 2])
    full = orc.input_rows(cfg, model, feats, ids)
    part = orc.input_rows(cfg, model, feats, ids, rows0=rows0)
    vis = rows0[(rows0 >= v0) & (rows0 < v1)]
    assert np.array_equal(part[vis], full[vis]) and np.array_equal(part[:v0], full[:v0]) and np.array_equal(part[v1:], full[v1:])
    rest = np.setdiff1d(np.arange(v0, v1), vis)
    assert np.all(part[rest] == 0.0) and np.any(full[rest] != 0.0)
    # brute force on one row: dot products in Python floats
    w = orc.widen_bf16(model["proj"]); x = orc.widen_bf16(feats[3])
    assert np.allclose(part[v0 + 3], [float(np.dot(w[n], x)) for n in range(cfg.hidden)], rtol=1e-12, atol=1e-12)
    # a cached step whose unselected feature rows are garbage gives the same result
    prev, cur, changed = synth.rerandomised_pair(cfg, 5, 13)
    params = orc.SelectParams(top_k=32, alpha_override=[0.5, 1.0])
    outs = []
    for poison in (False, True):
        cache = orc.new_cache(cfg)
        orc.step(cfg, model, cache, prev, feats, ids, params)
        sel = orc.select(cfg, cur, cache, params)
        f2 = feats.copy()
        if poison:
            skipped = np.setdiff1d(np.arange(v0, v1), sel.rows[0]) - v0
            assert len(skipped) > 0
            f2[skipped] = synth.f32_to_bf16(np.full((len(skipped), cfg.hidden), 1000.0, dtype=np.float32))
        outs.append(orc.step(cfg, model, cache, cur, f2, ids, params, selection=sel).logits)
    assert np.array_equal(outs[0], outs[1])


def test_rope_complex_form_and_relative_property():
    cfg = synth.tiny_config()
    cos, sin = synth.rope_tables(cfg)
    rng = np.random.default_rng(2)
    d, half = cfg.head_dim, cfg.head_dim // 2
    x = rng.standard_normal((5, 3, d))
    pos = np.array([0, 1, 7, 40, 79])
    y = orc.rope(x, pos, cos, sin)
    # complex form: (x_i + i x_{i+d/2}) * exp(i * pos * theta^(-2i/d))
    theta = cfg.rope_theta ** (-np.arange(half) * 2.0 / d)
    z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * pos[:, None, None] * theta[None, None, :])
    np.testing.assert_allclose(y[..., :half], z.real, atol=1e-6)      # tables are fp32
    np.testing.assert_allclose(y[..., half:], z.imag, atol=1e-6)
    np.testing.assert_array_equal(y[0], x[0])                         # position 0 is the identity
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-6)
    # <rope(q,m), rope(k,n)> depends on m-n only
    q, k = rng.standard_normal((1, 1, d)), rng.standard_normal((1, 1, d))
    def dot(m, n):
        return float(np.sum(orc.rope(q, np.array([m]), cos, sin) * orc.rope(k, np.array([n]), cos, sin)))
    assert abs(dot(9, 4) - dot(30, 25)) < 1e-5 and abs(dot(9, 4) - dot(5, 0)) < 1e-5
    assert abs(dot(9, 4) - dot(4, 9)) > 1e-3


def test_attention_rows_are_distributions_and_single_key_returns_value():
    cfg, model, ids, feats = _tiny()
    cache = orc.new_cache(cfg)
    hidden = orc.input_rows(cfg, model, feats, ids)
    before = hidden.copy()
    emitted = orc.layer_forward(cfg, model["layers"][0], cache.K[0], cache.V[0], hidden,
                                np.arange(cfg.seq_len), model["rope_cos"], model["rope_sin"])
    s = emitted.sum(axis=1)                     # mass the text rows put on the vision block
    assert np.all(s > 0) and np.all(s < 1) and np.all(emitted >= 0)
    # position 0 sees only itself: attention output is V[0]; check through the residual algebra
    lw = {k: orc.widen_bf16(v) for k, v in model["layers"][0].items()}
    x0 = before[0] + cache.V[0][0].reshape(-1) @ lw["wo"].T
    xn = orc.rms_norm(x0[None], lw["g_mlp"], cfg.rms_eps)[0]
    g = xn @ lw["w_gate"].T
    want = x0 + ((g / (1 + np.exp(-g))) * (xn @ lw["w_up"].T)) @ lw["w_down"].T
    np.testing.assert_allclose(hidden[0], want, atol=1e-12)


def test_emitted_attention_matches_textbook_softmax():
    """The emitted block equals rows of softmax(QK^T/sqrt(d)) restricted to (text query, vision key)."""
    cfg, model, ids, feats = _tiny()
    L = cfg.seq_len
    cache = orc.new_cache(cfg)
    hidden = orc.input_rows(cfg, model, feats, ids)
    h0 = torch.from_numpy(hidden[:L].copy())
    emitted = orc.layer_forward(cfg, model["layers"][0], cache.K[0], cache.V[0], hidden, np.arange(L),
                                model["rope_cos"], model["rope_sin"])
    lw = model["layers"][0]
    F = torch.nn.functional
    cos = torch.from_numpy(model["rope_cos"][:L].astype(np.float64)); sin = torch.from_numpy(model["rope_sin"][:L].astype(np.float64))
    xn = F.rms_norm(h0, (cfg.hidden,), _t(lw["g_attn"]), cfg.rms_eps)
    q = _torch_rope(F.linear(xn, _t(lw["wq"])).view(L, cfg.n_heads, cfg.head_dim), cos, sin)
    k = _torch_rope(F.linear(xn, _t(lw["wk"])).view(L, cfg.n_heads, cfg.head_dim), cos, sin)
    sc = torch.einsum("qhd,khd->hqk", q, k) / math.sqrt(cfg.head_dim)
    sc = sc.masked_fill(torch.triu(torch.ones(L, L, dtype=torch.bool), 1), float("-inf"))
    p = torch.softmax(sc, dim=-1)
    v0, v1 = cfg.n_text_pre, cfg.n_text_pre + cfg.n_vision
    want = p[:, v1:L, v0:v1].mean(dim=1).numpy()
    np.testing.assert_allclose(emitted, want, atol=1e-12)


def test_decode_pass_equals_longer_prefill():
    """Appending one token through the K/V cache gives the row a full causal pass over the
    longer sequence gives (Sec. 3.1, cache append)."""
    cfg, model, ids, feats = _tiny()
    L = cfg.seq_len
    cache = orc.new_cache(cfg)
    res = orc.step(cfg, model, cache, np.zeros((1, 112, 112, 3), np.uint8), feats, ids, orc.SelectParams())
    h = orc.input_rows(cfg, model, feats, ids)
    h[L] = orc.widen_bf16(model["embed"][int(res.tokens[0])])
    ht = torch.from_numpy(h[:L + 1].copy())
    cos = torch.from_numpy(model["rope_cos"][:L + 1].astype(np.float64)); sin = torch.from_numpy(model["rope_sin"][:L + 1].astype(np.float64))
    for l in range(cfg.n_layers):
        ht, _, _ = _torch_layer(cfg, model["layers"][l], ht, cos, sin)
    F = torch.nn.functional
    logits = F.linear(F.rms_norm(ht[L], (cfg.hidden,), _t(model["g_final"]), cfg.rms_eps), _t(model["lm_head"]))
    np.testing.assert_allclose(res.logits[1], logits.numpy(), atol=1e-9)
    assert int(torch.argmax(logits)) == int(res.tokens[1])
    logits0 = F.linear(F.rms_norm(ht[L - 1], (cfg.hidden,), _t(model["g_final"]), cfg.rms_eps), _t(model["lm_head"]))
    np.testing.assert_allclose(res.logits[0], logits0.numpy(), atol=1e-9)


def test_chunk_pass_equals_joint_forward_with_block_mask():
    """A chunk of action rows decoded in parallel behind a full prefill equals ONE forward of
    textbook layers over prompt + chunk under the mask "causal, except that chunk rows see the
    whole chunk": the prompt rows never see the chunk, so prefill-then-chunk and the joint pass
    are the same function.  Pins the mask, the positions of the chunk rows and the K/V append."""
    cfg, model, ids, feats = _tiny()
    L, n = cfg.seq_len, cfg.n_action
    act = synth.make_action_embed(cfg, 3)
    cache = orc.new_cache(cfg)
    res = orc.step_chunk(cfg, model, cache, np.zeros((1, 112, 112, 3), np.uint8), feats, ids, orc.SelectParams(), act)
    h = orc.input_rows(cfg, model, feats, ids)
    h[L:L + n] = orc.widen_bf16(act)
    ht = torch.from_numpy(h[:L + n].copy())
    cos = torch.from_numpy(model["rope_cos"][:L + n].astype(np.float64)); sin = torch.from_numpy(model["rope_sin"][:L + n].astype(np.float64))
    mask = torch.tril(torch.ones(L + n, L + n, dtype=torch.bool))
    mask[L:, L:] = True
    for l in range(cfg.n_layers):
        ht, k, v = _torch_layer(cfg, model["layers"][l], ht, cos, sin, mask=mask)
        np.testing.assert_allclose(cache.K[l][:L + n], k.numpy(), atol=1e-10)
        np.testing.assert_allclose(cache.V[l][:L + n], v.numpy(), atol=1e-10)
    F = torch.nn.functional
    logits = F.linear(F.rms_norm(ht[L:], (cfg.hidden,), _t(model["g_final"]), cfg.rms_eps), _t(model["lm_head"]))
    np.testing.assert_allclose(res.logits, logits.numpy(), atol=1e-9)
    assert torch.argmax(logits, dim=1).tolist() == res.tokens.tolist()
    # the mask matters: a purely causal pass gives other logits for every row but the last
    hc = torch.from_numpy(h[:L + n].copy())
    for l in range(cfg.n_layers):
        hc, _, _ = _torch_layer(cfg, model["layers"][l], hc, cos, sin)
    lc = F.linear(F.rms_norm(hc[L:], (cfg.hidden,), _t(model["g_final"]), cfg.rms_eps), _t(model["lm_head"])).numpy()
    assert np.abs(lc[:-1] - res.logits[:-1]).max() > 1e-6


def test_chunk_step_leaves_the_prompt_state_of_an_ordinary_step():
    """The chunk pass writes only behind the prompt: selection, prompt K/V, prompt hidden rows and the
    emitted text-to-vision attention of a chunk step equal those of an ordinary step on the same
    inputs, cold and cached."""
    cfg, model, ids, feats = _tiny()
    L = cfg.seq_len
    act = synth.make_action_embed(cfg, 3)
    prev, cur, _ = synth.rerandomised_pair(cfg, 0, 13)
    params = orc.SelectParams(top_k=32, alpha_override=[0.5, 1.0])
    ca, cb = orc.new_cache(cfg), orc.new_cache(cfg)
    for frame in (prev, cur):
        ra = orc.step(cfg, model, ca, frame, feats, ids, params)
        rb = orc.step_chunk(cfg, model, cb, frame, feats, ids, params, act)
        assert [r.tolist() for r in ra.selection.rows] == [r.tolist() for r in rb.selection.rows]
        np.testing.assert_array_equal(ca.K[:, :L], cb.K[:, :L])
        np.testing.assert_array_equal(ca.V[:, :L], cb.V[:, :L])
        np.testing.assert_array_equal(ra.hidden[:L], rb.hidden[:L])
        np.testing.assert_array_equal(ra.attn_tv, rb.attn_tv)
    assert rb.selection.M[1] < L


def _two_steps(cfg, model, ids, feats0, feats1, prev, cur, params, force_full=False):
    cache = orc.new_cache(cfg)
    orc.step(cfg, model, cache, prev, feats0, ids, params)
    return orc.step(cfg, model, cache, cur, feats1, ids, params, force_full=force_full), cache


def test_reuse_ratio_zero_equals_full_prefill():
    cfg, model, ids, feats = _tiny()
    prev, cur, _ = synth.rerandomised_pair(cfg, 0, 13)
    feats1 = synth.f32_to_bf16(np.random.default_rng(9).standard_normal((cfg.n_vision, cfg.hidden), dtype=np.float32))
    p0 = orc.SelectParams(top_k=32, alpha_override=[0.0] * cfg.n_layers)
    a, ca = _two_steps(cfg, model, ids, feats, feats1, prev, cur, p0)
    b, cb = _two_steps(cfg, model, ids, feats, feats1, prev, cur, p0, force_full=True)
    assert np.all(a.selection.M == cfg.seq_len) and a.selection.final_mask.sum() > 0
    np.testing.assert_array_equal(a.logits, b.logits)
    np.testing.assert_array_equal(ca.K, cb.K)
    np.testing.assert_array_equal(a.attn_tv, b.attn_tv)
    # and a cold step is a full prefill of the same inputs
    cold = orc.step(cfg, model, orc.new_cache(cfg), cur, feats1, ids, p0)
    np.testing.assert_array_equal(cold.logits, b.logits)


def test_identical_inputs_make_any_reuse_set_exact():
    """If nothing changed between two steps, reused K/V equal recomputed K/V, so the cached
    step equals the full step whatever is reused."""
    cfg, model, ids, feats = _tiny()
    prev, _, _ = synth.rerandomised_pair(cfg, 0, 13)
    for alpha in ([1.0, 1.0], [0.3, 0.8]):
        p = orc.SelectParams(top_k=40, alpha_override=alpha)
        a, ca = _two_steps(cfg, model, ids, feats, feats, prev, prev, p)
        b, cb = _two_steps(cfg, model, ids, feats, feats, prev, prev, p, force_full=True)
        assert a.selection.M[1] < cfg.seq_len
        np.testing.assert_allclose(a.logits, b.logits, atol=1e-12)
        np.testing.assert_allclose(ca.K, cb.K, atol=1e-12)
        assert list(a.tokens) == list(b.tokens)


def test_causality_prefix_before_first_change_is_exact():
    """Every position before the first changed input has K/V identical to full recomputation,
    and reused positions keep exactly the previous step's K/V (Algorithm 2)."""
    cfg, model, ids, feats = _tiny()
    prev, cur, changed = synth.rerandomised_pair(cfg, 0, 13)
    first = int(changed.min())
    feats1 = feats.copy()
    rng = np.random.default_rng(4)
    for v in changed:
        feats1[v] = synth.f32_to_bf16(rng.standard_normal(cfg.hidden, dtype=np.float32))
    p = orc.SelectParams(top_k=32, alpha_override=[1.0] * cfg.n_layers)
    cache = orc.new_cache(cfg)
    orc.step(cfg, model, cache, prev, feats, ids, p)
    K_before = cache.K.copy()
    a = orc.step(cfg, model, cache, cur, feats1, ids, p)
    b, cb = _two_steps(cfg, model, ids, feats, feats1, prev, cur, p, force_full=True)
    n_prefix = cfg.n_text_pre + first
    np.testing.assert_allclose(cache.K[:, :n_prefix], cb.K[:, :n_prefix], atol=1e-12)
    np.testing.assert_allclose(cache.V[:, :n_prefix], cb.V[:, :n_prefix], atol=1e-12)
    for l in range(cfg.n_layers):
        skipped = sorted(set(range(cfg.seq_len)) - set(a.selection.rows[l].tolist()))
        assert len(skipped) == int(a.selection.final_mask.sum()) > 0
        np.testing.assert_array_equal(cache.K[l][skipped], K_before[l][skipped])
    # the approximation is real: positions after the change differ from full recomputation
    late = [p_ for p_ in skipped if p_ > n_prefix]
    assert late and np.abs(cache.K[1][late] - cb.K[1][late]).max() > 1e-9      # stale layer-1 keys
    np.testing.assert_allclose(cache.K[0][:cfg.seq_len], cb.K[0][:cfg.seq_len], atol=1e-12)                # layer-0 K/V see only their own input
    assert np.abs(a.logits - b.logits).max() > 1e-9


def test_forced_tokens_are_fed_back():
    cfg, model, ids, feats = _tiny()
    frame = np.zeros((1, 112, 112, 3), np.uint8)
    free = orc.step(cfg, model, orc.new_cache(cfg), frame, feats, ids, orc.SelectParams())
    forced = free.tokens.copy(); forced[0] = (forced[0] + 1) % cfg.vocab
    r = orc.step(cfg, model, orc.new_cache(cfg), frame, feats, ids, orc.SelectParams(), forced_tokens=forced)
    np.testing.assert_array_equal(r.logits[0], free.logits[0])
    assert r.tokens[0] == free.tokens[0] and np.abs(r.logits[1] - free.logits[1]).max() > 1e-9
    assert np.all(r.margins >= 0)


def test_layer_major_composition_equals_step():
    """tests/oracle_compose.step_layer_major (each layer once: prefill rows, then the single rows) gives the
    bits of oracle.step when it is fed the same tokens, cold and cached."""
    import oracle_compose
    cfg, model, ids, feats = _tiny(4)
    prev, cur, _ = synth.rerandomised_pair(cfg, 4, 13)
    params = orc.SelectParams(top_k=32, alpha_override=[0.5, 1.0])
    ca, cb = orc.new_cache(cfg), orc.new_cache(cfg)
    for fr in (prev, cur):
        ra = orc.step(cfg, model, ca, fr, feats, ids, params)
        rb = oracle_compose.step_layer_major(cfg, model, cb, fr, feats, ids, params, forced_tokens=ra.tokens)
        assert np.array_equal(ra.logits, rb.logits) and np.array_equal(ra.tokens, rb.tokens)
        assert np.array_equal(ra.attn_tv, rb.attn_tv) and np.array_equal(ra.hidden, rb.hidden)
        assert np.array_equal(ca.K, cb.K) and np.array_equal(ca.V, cb.V)
    assert ra.selection.M[1] < cfg.seq_len



def _torch_bf16(t):
    return t.to(torch.bfloat16).double()


def test_round_bf16_matches_torch_conversion():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-30, 30, size=20000),
                        np.array([0.0, -0.0, 1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -9, -(1.0 + 2.0 ** -8),
                                  2.0 ** -133, 2.0 ** -134, 3.0e38, 3.4e38, np.inf, -np.inf])])
    got = orc.round_bf16(x)
    want = torch.from_numpy(x).to(torch.bfloat16).double().numpy()
    assert np.array_equal(got, want) and np.array_equal(np.signbit(got), np.signbit(want))
    assert got[20003] == 1.0 and got[20004] == 1.0 + 2.0 ** -6           # ties go to the even mantissa


def test_bf16_operand_setting_equals_torch_layer_with_torch_roundings():
    """operands="bf16": the same textbook layer, every matrix-product operand rounded by torch's own bf16 conversion."""
    cfg, model, ids, feats = _tiny(6)
    L = cfg.seq_len
    h0 = orc.input_rows(cfg, model, feats, ids)
    cos, sin = torch.from_numpy(model["rope_cos"][:L]).double(), torch.from_numpy(model["rope_sin"][:L]).double()
    K = np.zeros((cfg.max_seq, cfg.n_heads, cfg.head_dim)); V = np.zeros_like(K)
    hid = h0.copy()
    orc.layer_forward(cfg, model["layers"][0], K, V, hid, np.arange(L), model["rope_cos"], model["rope_sin"], operands="bf16")
    want, k, v = _torch_layer(cfg, model["layers"][0], torch.from_numpy(h0[:L]), cos, sin, rb=_torch_bf16)
    np.testing.assert_allclose(hid[:L], want.numpy(), rtol=0, atol=2e-3 * np.abs(want.numpy()).max())   # a rounding may flip where fp64 sums differ in the last bit
    assert np.median(np.abs(hid[:L] - want.numpy())) <= 1e-9 * np.abs(want.numpy()).max()
    assert np.array_equal(K[:L], orc.round_bf16(K[:L])) and np.array_equal(V[:L], orc.round_bf16(V[:L]))      # stored as bf16 values
    np.testing.assert_allclose(K[:L], k.numpy(), rtol=0, atol=2.0 ** -7 * np.abs(k.numpy()).max())
    # and the exact setting is a different function of the same inputs
    hid_x = h0.copy()
    Kx = np.zeros_like(K); Vx = np.zeros_like(V)
    orc.layer_forward(cfg, model["layers"][0], Kx, Vx, hid_x, np.arange(L), model["rope_cos"], model["rope_sin"])
    d = np.abs(hid_x[:L] - hid[:L]).max() / np.abs(hid_x[:L]).max()
    assert 1e-4 < d < 2e-2


def test_cost_of_bf16_operands_on_the_tiny_decoder():
    """Distance between the checker's two settings on the tiny decoder stacked to 2 and 8 layers: a bf16 computation
    is a different function from exact arithmetic, by a few 1e-3 of the largest logit at this width.  (On the 32-layer
    7B shape the same distance is measured in tests/test_gpu_parity.py, where the host is fast enough.)"""
    cfg8 = synth.tiny_config().with_layers(8)
    model = synth.make_model(cfg8, 9)
    ids = synth.make_prompt_ids(cfg8, 9)[0]
    feats = synth.f32_to_bf16(np.random.default_rng(10).standard_normal((cfg8.n_vision, cfg8.hidden), dtype=np.float32))
    frame = synth.rerandomised_pair(cfg8, 9, 0)[0]
    for nl in (2, 8):
        cfg = cfg8.with_layers(nl)
        m = dict(model, layers=model["layers"][:nl])
        ra = orc.step(cfg, m, orc.new_cache(cfg), frame, feats, ids, orc.SelectParams())
        rb = orc.step(cfg, m, orc.new_cache(cfg), frame, feats, ids, orc.SelectParams(), forced_tokens=ra.tokens, operands="bf16")
        dist = max(float(np.abs(rb.logits[i] - ra.logits[i]).max() / np.abs(ra.logits[i]).max()) for i in range(cfg.n_action))
        assert 1e-4 < dist < 2e-2, (nl, dist)


def test_pruned_tokens_match_a_brute_force_sort():
    rng = np.random.default_rng(3)
    score = np.round(rng.random(40), 1)                       # many ties
    for n_keep in (0, 1, 7, 39, 40, 50):
        keep = orc.pruned_vision_tokens(score, n_keep)
        order = np.lexsort((np.arange(40), -score))          # by score descending, then index ascending
        want = np.zeros(40, dtype=bool); want[order[:min(n_keep, 40)]] = True
        assert np.array_equal(keep, want)


def test_pruned_step_special_cases_and_textbook_model_on_the_reduced_sequence():
    """step_pruned: keeping every token (or pruning behind the last layer) is the plain step, bit for bit; and with
    tokens dropped after layer 0, layer 1 equals a textbook layer run on the REDUCED sequence (dropped tokens removed,
    the others at their original rotary positions)."""
    cfg, model, ids, feats = _tiny(7)
    frame = synth.rerandomised_pair(cfg, 7, 0)[0]
    L, v0, lv = cfg.seq_len, cfg.n_text_pre, cfg.n_vision
    full = orc.step(cfg, model, orc.new_cache(cfg), frame, feats, ids, orc.SelectParams())
    for args in ((1, lv), (cfg.n_layers, 10)):
        same = orc.step_pruned(cfg, model, orc.new_cache(cfg), frame, feats, ids, *args)
        assert np.array_equal(same.logits, full.logits) and np.array_equal(same.tokens, full.tokens)
    n_keep = 24
    cache = orc.new_cache(cfg)
    res = orc.step_pruned(cfg, model, cache, frame, feats, ids, 1, n_keep)
    assert list(res.selection.M) == [L, L - (lv - n_keep)]
    assert not np.array_equal(res.logits, full.logits)
    # layer 0 by the textbook layer, scores from its softmax, kept set by sorting
    h0 = torch.from_numpy(orc.input_rows(cfg, model, feats, ids)[:L])
    cos, sin = torch.from_numpy(model["rope_cos"][:L]).double(), torch.from_numpy(model["rope_sin"][:L]).double()
    h1, k0, v0_ = _torch_layer(cfg, model["layers"][0], h0, cos, sin)
    xn = torch.nn.functional.rms_norm(h0, (cfg.hidden,), _t(model["layers"][0]["g_attn"]), cfg.rms_eps)
    q = _torch_rope(torch.nn.functional.linear(xn, _t(model["layers"][0]["wq"])).view(L, cfg.n_heads, cfg.head_dim), cos, sin)
    sc = torch.einsum("qhd,khd->hqk", q, k0) / math.sqrt(cfg.head_dim)
    sc = sc.masked_fill(~torch.tril(torch.ones(L, L, dtype=torch.bool)), float("-inf"))
    p = torch.softmax(sc, dim=-1)
    score = p[:, v0 + lv:L, v0:v0 + lv].mean(dim=1).mean(dim=0).numpy()
    kept = np.zeros(lv, dtype=bool); kept[np.lexsort((np.arange(lv), -score))[:n_keep]] = True
    assert np.array_equal(~res.selection.final_mask, kept)
    rows = np.asarray([p_ for p_ in range(L) if not (v0 <= p_ < v0 + lv and not kept[p_ - v0])])
    assert np.array_equal(res.selection.rows[1], rows)
    h2, k1, v1 = _torch_layer(cfg, model["layers"][1], h1[rows], cos[rows], sin[rows])
    np.testing.assert_allclose(res.hidden[rows], h2.numpy(), rtol=1e-9, atol=1e-9)
    np.testing.assert_allclose(cache.K[1][rows], k1.numpy(), rtol=1e-9, atol=1e-9)
    np.testing.assert_allclose(cache.V[1][rows], v1.numpy(), rtol=1e-9, atol=1e-9)
    # the first logits row is the lm_head of the last reduced row
    xf = torch.nn.functional.rms_norm(h2[-1:], (cfg.hidden,), _t(model["g_final"]), cfg.rms_eps)
    np.testing.assert_allclose(res.logits[0], torch.nn.functional.linear(xf, _t(model["lm_head"]))[0].numpy(), rtol=1e-9, atol=1e-9)
