"""Pins for the selection half of the CPU checker (Sec. 3.2-3.4, Algorithm 1).

Each test fixes the checker to something outside itself: exact closed forms, exact rational
arithmetic, a textbook library routine, brute force on tiny inputs, a hand-worked example,
or an invariant the paper states.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import vla_cache_oracle as orc
from paper_2502_02175_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _frames(grid, patch, fill=0, cams=1):
    hw = grid * patch
    return np.full((cams, hw, hw, 3), fill, dtype=np.uint8)


# ----------------------------------------------------------------------------- Eq. (sim)
def test_similarity_closed_forms():
    grid, patch = 2, 14
    rng = np.random.default_rng(0)
    a = rng.integers(1, 120, size=(1, 28, 28, 3), dtype=np.uint8)
    # identical frames: exactly 1
    assert np.all(orc.patch_similarity(a, a, grid, patch) == 1.0)
    # b = 2a without clipping: na*nb is a perfect square, cosine is exactly 1
    assert np.all(orc.patch_similarity((2 * a).astype(np.uint8), a, grid, patch) == 1.0)
    # disjoint channel support: exactly 0
    r = np.zeros_like(a); r[..., 0] = a[..., 0]
    g = np.zeros_like(a); g[..., 1] = a[..., 1]
    assert np.all(orc.patch_similarity(r, g, grid, patch) == 0.0)
    # zero-norm readings
    z = np.zeros_like(a)
    assert np.all(orc.patch_similarity(z, z, grid, patch) == 1.0)
    assert np.all(orc.patch_similarity(a, z, grid, patch) == 0.0)


def test_similarity_matches_exact_rational_and_library():
    import torch
    cfg = synth.tiny_config()
    prev, cur, _ = synth.rerandomised_pair(cfg, 3, 20)
    sim = orc.patch_similarity(cur, prev, cfg.grid, cfg.patch)
    p = cfg.patch
    for idx in range(cfg.n_vision):
        i, j = divmod(idx, cfg.grid)
        a = [int(x) for x in cur[0, i * p:(i + 1) * p, j * p:(j + 1) * p, :].reshape(-1)]
        b = [int(x) for x in prev[0, i * p:(i + 1) * p, j * p:(j + 1) * p, :].reshape(-1)]
        dot = sum(x * y for x, y in zip(a, b))
        na, nb = sum(x * x for x in a), sum(y * y for y in b)
        # sim^2 must equal dot^2/(na*nb) to within two roundings
        exact_sq = Fraction(dot * dot, na * nb)
        assert abs(Fraction(sim[idx]) ** 2 - exact_sq) <= exact_sq * Fraction(4, 2 ** 52)
        ta = torch.tensor(a, dtype=torch.float64); tb = torch.tensor(b, dtype=torch.float64)
        lib = torch.nn.functional.cosine_similarity(ta, tb, dim=0).item()
        assert abs(lib - sim[idx]) < 1e-12


def test_similarity_patch_layout():
    """Changing one pixel of block-row i, block-column j, camera c moves exactly token c*N*N+i*N+j."""
    grid, patch = 4, 14
    base = np.random.default_rng(1).integers(1, 255, size=(2, 56, 56, 3), dtype=np.uint8)
    for cam, i, j, dy, dx, ch in [(0, 0, 3, 0, 0, 0), (1, 2, 1, 13, 13, 2), (0, 3, 0, 5, 7, 1)]:
        cur = base.copy()
        y, x = i * patch + dy, j * patch + dx
        cur[cam, y, x, ch] = np.uint8(255 - int(cur[cam, y, x, ch]))
        sim = orc.patch_similarity(cur, base, grid, patch)
        changed = np.nonzero(sim != 1.0)[0]
        assert list(changed) == [cam * 16 + i * 4 + j]


# ----------------------------------------------------------------------------- Eq. (topk)
def _brute_topk(sim, tau, k):
    pairs = sorted(((-s, v) for v, s in enumerate(sim) if s >= tau))
    return sorted(v for _, v in pairs[:k])


@pytest.mark.parametrize("seed", range(20))
def test_topk_matches_brute_force(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 24))
    sim = rng.choice(np.array([0.2, 0.5, 0.9, 0.996, 0.997, 1.0]), size=n)   # many ties
    tau = float(rng.choice([0.0, 0.5, 0.996, 1.0]))
    k = int(rng.integers(0, n + 2))
    mask = orc.static_tokens(sim, tau, k)
    assert sorted(np.nonzero(mask)[0]) == _brute_topk(sim, tau, k)


def test_topk_threshold_inclusive_and_tie_rule():
    sim = np.array([1.0, 0.996, 0.9959999, 1.0, 1.0])
    assert list(orc.static_tokens(sim, 0.996, 10)) == [True, True, False, True, True]
    assert list(orc.static_tokens(sim, 0.996, 2)) == [True, False, False, True, False]   # ties -> lower index


def test_tiny_config_tie_case():
    """51 of 64 patches are bit-identical (similarity exactly 1); top-k 32 keeps the 32 lowest ids."""
    cfg = synth.tiny_config()
    prev, cur, changed = synth.rerandomised_pair(cfg, 0, 13)
    sim = orc.patch_similarity(cur, prev, cfg.grid, cfg.patch)
    unchanged = [v for v in range(64) if v not in set(changed.tolist())]
    assert all(sim[v] == 1.0 for v in unchanged) and all(sim[v] < 0.9 for v in changed)
    mask = orc.static_tokens(sim, 0.996, 32)
    assert sorted(np.nonzero(mask)[0]) == unchanged[:32]


# ----------------------------------------------------------------------------- Sec. 3.3
def test_task_relevance_is_two_means():
    rng = np.random.default_rng(5)
    a = rng.random((3, 4, 6)).astype(np.float32)
    S_layer, S = orc.task_relevance(a)
    np.testing.assert_allclose(S_layer, a.astype(np.float64).mean(axis=1), rtol=1e-14)
    np.testing.assert_allclose(S, a.astype(np.float64).mean(axis=(0, 1)), rtol=1e-14)
    _, S2 = orc.task_relevance(a, layer_mask=[False, True, False])
    np.testing.assert_allclose(S2, a[1].astype(np.float64).mean(axis=0), rtol=1e-14)


@pytest.mark.parametrize("seed", range(10))
def test_task_tokens_match_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(2, 30))
    S = rng.choice(np.array([0.0, 0.01, 0.02, 0.3]), size=n)
    tau_task = float(rng.choice([0.0, 0.2, 0.5, 0.7, 1.0]))
    n_task = n - math.floor(tau_task * n)
    want = sorted(v for _, v in sorted((-s, v) for v, s in enumerate(S))[:n_task])
    assert sorted(np.nonzero(orc.task_relevant_tokens(S, tau_task, 0))[0]) == want
    assert list(orc.task_relevant_tokens(S, 0.02, 1)) == [bool(s >= 0.02) for s in S]


def test_eviction_is_set_difference():
    st = np.array([1, 1, 0, 0, 1], dtype=bool)
    tk = np.array([0, 1, 1, 0, 0], dtype=bool)
    assert list(orc.reusable_tokens(st, tk)) == [True, False, False, False, True]


# ----------------------------------------------------------------------------- Sec. 3.4
def test_entropy_closed_forms():
    lv = 16
    assert abs(orc.attention_entropy(np.full(lv, 0.01)) - math.log(lv)) < 1e-14
    onehot = np.zeros(lv); onehot[3] = 0.2
    assert orc.attention_entropy(onehot) == 0.0
    two = np.zeros(lv); two[[1, 7]] = 0.3
    assert abs(orc.attention_entropy(two) - math.log(2)) < 1e-14
    assert orc.attention_entropy(np.zeros(lv)) == math.log(lv)
    S_layer = np.full((5, lv), 0.03)
    E, R, alpha, abar = orc.reuse_ratios(S_layer, 3.0)
    assert np.allclose(E, math.log(lv)) and np.all(np.abs(R) < 1e-15) and np.all(abar < 1e-14)


def test_reuse_ratio_hand_example():
    """4 vision tokens, 2 layers, worked by hand (values in tests/golden/entropy_example.txt).

    Layer 1 mean attention (0.1,0.2,0.3,0.4)/1, layer 2 (0.7,0.1,0.1,0.1).
    E0 = ln 4 = 1.3862943611198906
    E1 = -(0.1 ln 0.1 + 0.2 ln 0.2 + 0.3 ln 0.3 + 0.4 ln 0.4) = 1.2798542258336676
    E2 = -(0.7 ln 0.7 + 3*0.1 ln 0.1)                         = 0.9404479886553264
    R1 = (E0-E1)/E0 = 0.07678032766449214, R2 = (E1-E2)/E1 = 0.2651913243926352
    k = 2: alpha1 = 0.15356065532898427, alpha2 = min(2*(R1+R2),1) = 0.6839433041142546
    """
    vals = {}
    with open(os.path.join(GOLDEN, "entropy_example.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    S_layer = np.array([[0.1, 0.2, 0.3, 0.4], [0.7, 0.1, 0.1, 0.1]]) * 0.5   # scale must not matter
    E, R, alpha, abar = orc.reuse_ratios(S_layer, 2.0)
    for name, got in [("E0", E[0]), ("E1", E[1]), ("E2", E[2]), ("R1", R[0]), ("R2", R[1]),
                      ("alpha1", alpha[0]), ("alpha2", alpha[1])]:
        assert abs(got - vals[name]) < 1e-12, name
    _, _, alpha_big, _ = orc.reuse_ratios(S_layer, 10.0)
    assert alpha_big[1] == 1.0                                    # min(., 1)
    _, _, alpha_neg, abar_neg = orc.reuse_ratios(S_layer[::-1].copy(), 2.0)
    assert alpha_neg[1] >= 0.0 and abar_neg[1] >= abar_neg[0]     # clamp and running max


def _warm_cache(cfg, prev, attn):
    c = orc.new_cache(cfg)
    c.prev_frames, c.attn_tv, c.warm = prev, attn, True
    return c


def test_select_invariants_and_monotonicity():
    """Nested reuse sets inside P_final; |P_final| grows with k and with tau_task
    (the paper's sensitivity tables: larger k / larger tau_task give more reuse)."""
    cfg = synth.llama7b_config(n_layers=6)
    ep = synth.make_episode(cfg, 11, 2)
    attn = synth.scripted_attention(cfg, 11, hot_tokens=ep.touched[1])
    cache = _warm_cache(cfg, ep.frames[0], attn)
    last = -1
    for k in (0, 20, 50, 100, 180, 256):
        sel = orc.select(cfg, ep.frames[1], cache, orc.SelectParams(top_k=k, k_ent=2.0))
        n_final = int(sel.final_mask.sum())
        assert n_final >= last; last = n_final
        assert np.all((sel.alpha >= 0) & (sel.alpha <= 1)) and np.all(np.diff(sel.alpha_bar) >= 0)
        assert sel.static_mask.sum() <= k and not np.any(sel.final_mask & sel.task_mask)
        prev_set = set()
        for l in range(cfg.n_layers):
            skipped = set(range(cfg.seq_len)) - set(sel.rows[l].tolist())
            assert prev_set <= skipped
            assert all(sel.final_mask[p - cfg.n_text_pre] for p in skipped)
            assert len(skipped) == sel.n_reuse[l] == math.floor(sel.alpha_bar[l] * n_final)
            assert list(sel.rows[l]) == sorted(sel.rows[l]) and sel.M[l] == len(sel.rows[l])
            prev_set = skipped
    last = -1
    for tt in (0.0, 0.2, 0.5, 0.7, 1.0):
        sel = orc.select(cfg, ep.frames[1], cache, orc.SelectParams(top_k=100, tau_task=tt))
        n_final = int(sel.final_mask.sum())
        assert n_final >= last; last = n_final
    # least task-relevant tokens are reused first
    sel = orc.select(cfg, ep.frames[1], cache, orc.SelectParams(top_k=100, alpha_override=[0.5] * 6))
    order = sel.reuse_order
    assert all((sel.S[a], a) < (sel.S[b], b) for a, b in zip(order[:-1], order[1:]))
    skipped = set(range(cfg.seq_len)) - set(sel.rows[0].tolist())
    assert skipped == {cfg.n_text_pre + int(v) for v in order[:len(order) // 2]}


def test_cold_cache_and_force_full_recompute_everything():
    cfg = synth.tiny_config()
    prev, cur, _ = synth.rerandomised_pair(cfg, 0, 13)
    sel = orc.select(cfg, cur, orc.new_cache(cfg), orc.SelectParams())
    assert all(list(r) == list(range(cfg.seq_len)) for r in sel.rows)
    attn = synth.scripted_attention(cfg, 0)
    sel = orc.select(cfg, cur, _warm_cache(cfg, prev, attn), orc.SelectParams(), force_full=True)
    assert np.all(sel.M == cfg.seq_len)


def test_paper_default_hyperparameters():
    """Appendix "Experimental Settings": tau 0.996, top-k 100, tau_task 0.5, 256 vision tokens, 7 action tokens."""
    vals = {}
    with open(os.path.join(GOLDEN, "paper_defaults.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split("=")
                vals[k.strip()] = float(v)
    p = orc.SelectParams()
    assert (p.tau, p.top_k, p.tau_task) == (vals["tau"], int(vals["top_k"]), vals["tau_task"])
    cfg = synth.llama7b_config()
    assert cfg.n_vision == int(vals["vision_tokens"]) and cfg.n_action == int(vals["action_tokens"])


def test_noisy_regime_needs_the_lower_threshold():
    """Appendix "Experimental Settings": on the real robot the similarity threshold is lowered to 0.85 to
    absorb sensor noise.  With Gaussian pixel noise of sigma 12 on a static background an untouched patch has
    cosine similarity about 1 - sigma^2 / E[x^2] ~ 0.993: under the default 0.996 almost none counts as static,
    under 0.85 every untouched patch does.  Raw-pixel vectors are non-negative, so even a patch a blob moved
    over stays near 0.9 and passes 0.85 too; there the top-k cap does the filtering, keeping the most similar."""
    cfg = synth.llama7b_config(n_layers=1)
    ep = synth.make_episode(cfg, 11, 3, n_blobs=3, noise_sigma=12.0)
    sim = orc.patch_similarity(ep.frames[2], ep.frames[1], cfg.grid, cfg.patch)
    touched = np.zeros(cfg.n_vision, dtype=bool)
    touched[np.asarray(ep.touched[2], dtype=np.int64)] = True
    untouched = ~touched
    assert untouched.sum() > 150 and touched.sum() > 20
    assert np.all(np.abs(sim - 0.85) >= 1e-5) and np.all(np.abs(sim - 0.996) >= 1e-5)
    expect = 1.0 - 144.0 / (255.0 ** 2 / 3.0)                     # E[x^2] of uniform bytes ~ 255^2 / 3
    assert abs(float(np.median(sim[untouched])) - expect) < 2e-3
    assert float(np.median(sim[touched])) < float(np.median(sim[untouched])) - 0.02
    strict = orc.static_tokens(sim, 0.996, cfg.n_vision)
    loose = orc.static_tokens(sim, 0.85, cfg.n_vision)
    assert strict[untouched].mean() < 0.10
    assert loose[untouched].all()
    capped = orc.static_tokens(sim, 0.85, 100)
    assert capped.sum() == 100 and sim[capped].min() >= np.sort(sim)[-100]
    assert capped[touched].sum() <= 0.2 * touched.sum() + 10


def test_similarity_of_real_valued_frames():
    """patch_similarity_values: closed forms, the integer path on byte frames, and torch's cosine_similarity."""
    import torch
    cfg = synth.tiny_config()
    prev, cur, changed = synth.rerandomised_pair(cfg, 11, 13)
    # on byte frames the two functions are the same quantity
    a = orc.patch_similarity(cur, prev, cfg.grid, cfg.patch)
    b = orc.patch_similarity_values(cur.astype(np.float64), prev.astype(np.float64), cfg.grid, cfg.patch)
    np.testing.assert_allclose(b, a, rtol=0, atol=1e-15)
    # normalised frames: centred pixels change the values (and allow negative similarities)
    x = (cur.astype(np.float64) / 255.0 - 0.5) / 0.25
    y = (prev.astype(np.float64) / 255.0 - 0.5) / 0.25
    s = orc.patch_similarity_values(x, y, cfg.grid, cfg.patch)
    unchanged = np.setdiff1d(np.arange(cfg.n_vision), changed)
    assert np.all(s[unchanged] == 1.0) and np.all(np.abs(s[changed]) < 0.2)
    p = cfg.patch
    for v in (0, int(changed[0]), cfg.n_vision - 1):
        i, j = divmod(v, cfg.grid)
        ta = torch.from_numpy(x[0, i * p:(i + 1) * p, j * p:(j + 1) * p, :].reshape(1, -1))
        tb = torch.from_numpy(y[0, i * p:(i + 1) * p, j * p:(j + 1) * p, :].reshape(1, -1))
        assert abs(float(torch.nn.functional.cosine_similarity(ta, tb)) - s[v]) < 1e-12
    assert np.all(orc.patch_similarity_values(x, -x, cfg.grid, cfg.patch) == -1.0)
    z = np.zeros_like(x)
    assert np.all(orc.patch_similarity_values(z, z, cfg.grid, cfg.patch) == 1.0)
    assert np.all(orc.patch_similarity_values(x, z, cfg.grid, cfg.patch) == 0.0)
    # select() on values: same sets as on bytes when only the scale changes (cosine is scale-free)
    cache = orc.new_cache(cfg)
    cache.warm, cache.prev_frames = True, prev
    cache.attn_tv = synth.scripted_attention(cfg, 11).astype(np.float64)
    want = orc.select(cfg, cur, cache, orc.SelectParams(top_k=32))
    cache.prev_frames = prev.astype(np.float64) / 255.0
    got = orc.select(cfg, cur.astype(np.float64) / 255.0, cache, orc.SelectParams(top_k=32), frame_values=True)
    assert np.array_equal(got.final_mask, want.final_mask) and np.array_equal(got.M, want.M)
