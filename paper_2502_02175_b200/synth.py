"""Seeded synthetic inputs for the cached-prefill path.

Everything here is data generation: random weights of a Llama-2-shaped decoder,
camera frames with a static background and moving blobs, vision features, prompt
ids, rotary tables and scripted attention tensors.  None of the method's
arithmetic (similarity, selection, attention, ...) is implemented here, so the
same arrays can be handed to the CUDA library and to the CPU checker.

Floating-point model data is produced as bf16 bit patterns (``uint16``); use
``bf16_to_f32`` / ``bf16_to_f64`` to widen them.  All draws come from
``numpy.random.default_rng(seed)``.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Optional, Tuple

import numpy as np


# --------------------------------------------------------------------------- #
# number formats
# --------------------------------------------------------------------------- #
def f32_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_to_f32(b).astype(np.float64)


# --------------------------------------------------------------------------- #
# configuration
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class ModelConfig:
    """Shape of the decoder and of the token sequence.

    The sequence is ``[n_text_pre text][n_cams*grid*grid vision][n_text_post text]``;
    each camera frame is a ``grid*patch`` square of uint8 RGB pixels.
    """
    n_layers: int
    hidden: int
    n_heads: int
    head_dim: int
    ffn: int
    vocab: int
    n_cams: int
    grid: int
    patch: int
    n_text_pre: int
    n_text_post: int
    n_action: int = 7
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def n_vision(self) -> int:
        return self.n_cams * self.grid * self.grid

    @property
    def seq_len(self) -> int:
        return self.n_text_pre + self.n_vision + self.n_text_post

    @property
    def n_text(self) -> int:
        return self.n_text_pre + self.n_text_post

    @property
    def max_seq(self) -> int:
        """Prefill length plus room for the K/V of the action rows (one per action token: the fed-back
        tokens use all but the last, a chunk decoded in parallel uses all)."""
        return self.seq_len + self.n_action

    @property
    def frame_hw(self) -> int:
        return self.grid * self.patch

    def with_layers(self, n_layers: int) -> "ModelConfig":
        return dataclasses.replace(self, n_layers=n_layers)


def tiny_config() -> ModelConfig:
    """2-layer decoder, hidden 256, 4x64 heads, FFN 688, 16 text + 64 vision tokens."""
    return ModelConfig(n_layers=2, hidden=256, n_heads=4, head_dim=64, ffn=688, vocab=1024,
                       n_cams=1, grid=8, patch=14, n_text_pre=1, n_text_post=15)


def llama7b_config(n_layers: int = 32, n_cams: int = 1, n_text_post: int = 33) -> ModelConfig:
    """Llama-2-7B shape: hidden 4096, 32x128 heads, FFN 11008, vocab 32000, 16x16 patches."""
    return ModelConfig(n_layers=n_layers, hidden=4096, n_heads=32, head_dim=128, ffn=11008,
                       vocab=32000, n_cams=n_cams, grid=16, patch=14, n_text_pre=1,
                       n_text_post=n_text_post)


def dual_camera_config(n_layers: int = 32) -> ModelConfig:
    """Two cameras (2x256 vision tokens) + 40 prompt tokens."""
    return llama7b_config(n_layers=n_layers, n_cams=2, n_text_post=39)


# --------------------------------------------------------------------------- #
# model weights
# --------------------------------------------------------------------------- #
LAYER_MATRICES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def layer_shapes(cfg: ModelConfig) -> Dict[str, Tuple[int, int]]:
    qd = cfg.n_heads * cfg.head_dim
    return {"wq": (qd, cfg.hidden), "wk": (qd, cfg.hidden), "wv": (qd, cfg.hidden),
            "wo": (cfg.hidden, qd), "w_gate": (cfg.ffn, cfg.hidden),
            "w_up": (cfg.ffn, cfg.hidden), "w_down": (cfg.hidden, cfg.ffn)}


def _normal_bf16(rng: np.random.Generator, shape, std: float, mean: float = 0.0) -> np.ndarray:
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(-1)
    n = flat.shape[0]
    chunk = 1 << 24
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        v = rng.standard_normal(e - s, dtype=np.float32)
        v *= np.float32(std)
        if mean != 0.0:
            v += np.float32(mean)
        flat[s:e] = f32_to_bf16(v)
    return out


def rope_tables(cfg: ModelConfig) -> Tuple[np.ndarray, np.ndarray]:
    """cos / sin of ``pos * theta**(-2i/d)`` for ``i < d/2``, made in fp64 and stored fp32."""
    half = cfg.head_dim // 2
    inv = cfg.rope_theta ** (-np.arange(half, dtype=np.float64) * 2.0 / cfg.head_dim)
    ang = np.arange(cfg.max_seq, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def make_model(cfg: ModelConfig, seed: int) -> Dict[str, object]:
    """Random-init weights: matrices N(0, 0.02), norm gains 1 + N(0, 0.1); all bf16 patterns.

    Returns ``{"layers": [ {name: uint16 [out,in]} ], "embed", "proj", "g_final",
    "lm_head", "rope_cos", "rope_sin"}``; matrices are ``[out_features, in_features]``.
    """
    rng = np.random.default_rng(seed)
    layers: List[Dict[str, np.ndarray]] = []
    shapes = layer_shapes(cfg)
    for _ in range(cfg.n_layers):
        lw = {name: _normal_bf16(rng, shapes[name], 0.02) for name in LAYER_MATRICES}
        lw["g_attn"] = _normal_bf16(rng, (cfg.hidden,), 0.1, 1.0)
        lw["g_mlp"] = _normal_bf16(rng, (cfg.hidden,), 0.1, 1.0)
        layers.append(lw)
    cos, sin = rope_tables(cfg)
    return {
        "layers": layers,
        "embed": _normal_bf16(rng, (cfg.vocab, cfg.hidden), 0.02),
        "proj": _normal_bf16(rng, (cfg.hidden, cfg.hidden), 0.02),
        "g_final": _normal_bf16(rng, (cfg.hidden,), 0.1, 1.0),
        "lm_head": _normal_bf16(rng, (cfg.vocab, cfg.hidden), 0.02),
        "rope_cos": cos,
        "rope_sin": sin,
    }


def make_prompt_ids(cfg: ModelConfig, seed: int, batch: int = 1) -> np.ndarray:
    """Random token ids ``[batch, n_text]`` (pre-vision tokens first, then post-vision)."""
    rng = np.random.default_rng(seed + 7919)
    return rng.integers(0, cfg.vocab, size=(batch, cfg.n_text), dtype=np.int32)


def make_action_embed(cfg: ModelConfig, seed: int) -> np.ndarray:
    """Placeholder embeddings ``[n_action, hidden]`` (bf16 bits) of the action rows that a chunk
    decoded in parallel starts from; same distribution as the token embeddings."""
    rng = np.random.default_rng(seed + 15485863)
    return _normal_bf16(rng, (cfg.n_action, cfg.hidden), 0.02)


def make_hidden(cfg: ModelConfig, seed: int, batch: int = 1, std: float = 1.0) -> np.ndarray:
    """Random bf16 hidden states ``[batch, seq_len, hidden]`` for single-layer cases."""
    rng = np.random.default_rng(seed + 104729)
    return _normal_bf16(rng, (batch, cfg.seq_len, cfg.hidden), std)


# --------------------------------------------------------------------------- #
# camera frames
# --------------------------------------------------------------------------- #
def _patch_slices(cfg: ModelConfig, idx: int) -> Tuple[slice, slice]:
    i, j = divmod(idx, cfg.grid)
    p = cfg.patch
    return slice(i * p, (i + 1) * p), slice(j * p, (j + 1) * p)


def rerandomised_pair(cfg: ModelConfig, seed: int, n_changed: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Two frames ``[n_cams,H,W,3]``: uniform random bytes; the second equals the first
    except ``n_changed`` patches (per camera) redrawn.  Returns (prev, cur, changed ids)."""
    rng = np.random.default_rng(seed)
    hw = cfg.frame_hw
    prev = rng.integers(0, 256, size=(cfg.n_cams, hw, hw, 3), dtype=np.uint8)
    cur = prev.copy()
    changed = []
    for c in range(cfg.n_cams):
        ids = np.sort(rng.choice(cfg.grid * cfg.grid, size=n_changed, replace=False))
        for idx in ids:
            ys, xs = _patch_slices(cfg, int(idx))
            cur[c, ys, xs, :] = rng.integers(0, 256, size=(cfg.patch, cfg.patch, 3), dtype=np.uint8)
            changed.append(c * cfg.grid * cfg.grid + int(idx))
    return prev, cur, np.asarray(changed, dtype=np.int64)


@dataclass
class Episode:
    """A synthetic camera stream plus the vision features that go with it."""
    frames: np.ndarray        # uint8 [n_steps, n_cams, H, W, 3]
    feats: np.ndarray         # uint16 (bf16) [n_steps, n_vision, hidden]
    touched: List[np.ndarray]  # per step: vision-token ids whose pixels were altered on purpose


def _blob_touch(cfg: ModelConfig, boxes: List[Tuple[int, int, int]]) -> np.ndarray:
    """Grid cells overlapped by any of the square boxes (y, x, size)."""
    hit = np.zeros((cfg.grid, cfg.grid), dtype=bool)
    p = cfg.patch
    for (y, x, s) in boxes:
        i0, i1 = max(y, 0) // p, min(y + s - 1, cfg.frame_hw - 1) // p
        j0, j1 = max(x, 0) // p, min(x + s - 1, cfg.frame_hw - 1) // p
        hit[i0:i1 + 1, j0:j1 + 1] = True
    return hit.reshape(-1)


def make_episode(cfg: ModelConfig, seed: int, n_steps: int, n_blobs: Optional[int] = None,
                 blob: int = 48, noise_sigma: float = 2.0,
                 changed_fraction: Optional[List[float]] = None) -> Episode:
    """Static uniform-noise background with moving flat-colour square blobs.

    Camera ``c`` follows ``changed_fraction[c]`` if given (that fraction of its patches is
    redrawn every step instead of blobs moving); otherwise ``n_blobs`` (default: drawn from
    1..3) blobs of side ``blob`` move 4-8 px per step along each axis and bounce at the
    border.  Every frame gets fresh Gaussian pixel noise of ``noise_sigma`` (clipped).
    Vision features are N(0,1); between steps a token's row is redrawn if its patch was
    touched on purpose, else carried over with N(0, 1e-3) jitter.
    """
    rng = np.random.default_rng(seed)
    hw, g2 = cfg.frame_hw, cfg.grid * cfg.grid
    frames = np.empty((n_steps, cfg.n_cams, hw, hw, 3), dtype=np.uint8)
    feats = np.empty((n_steps, cfg.n_vision, cfg.hidden), dtype=np.uint16)
    touched: List[np.ndarray] = []

    background = rng.integers(0, 256, size=(cfg.n_cams, hw, hw, 3)).astype(np.float32)
    blobs = []   # per camera: list of [y, x, vy, vx, colour]
    for c in range(cfg.n_cams):
        cam_blobs = []
        if changed_fraction is None or changed_fraction[c] is None:
            nb = int(rng.integers(1, 4)) if n_blobs is None else n_blobs
            for _ in range(nb):
                y, x = (int(v) for v in rng.integers(0, hw - blob, size=2))
                vy, vx = (int(v) * (1 if rng.random() < 0.5 else -1) for v in rng.integers(4, 9, size=2))
                colour = rng.integers(0, 256, size=3).astype(np.float32)
                cam_blobs.append([y, x, vy, vx, colour])
        blobs.append(cam_blobs)

    cur_feat = rng.standard_normal((cfg.n_vision, cfg.hidden), dtype=np.float32)
    for t in range(n_steps):
        hit_all = np.zeros(cfg.n_vision, dtype=bool)
        for c in range(cfg.n_cams):
            frac = None if changed_fraction is None else changed_fraction[c]
            if frac is not None:
                if t > 0:
                    ids = rng.choice(g2, size=int(round(frac * g2)), replace=False)
                    for idx in ids:
                        ys, xs = _patch_slices(cfg, int(idx))
                        background[c, ys, xs, :] = rng.integers(0, 256, size=(cfg.patch, cfg.patch, 3))
                        hit_all[c * g2 + int(idx)] = True
                img = background[c].copy()
            else:
                img = background[c].copy()
                boxes = []
                for b in blobs[c]:
                    if t > 0:
                        boxes.append((b[0], b[1], blob))          # area being uncovered
                        for ax, v in ((0, 2), (1, 3)):
                            b[ax] += b[v]
                            if b[ax] < 0 or b[ax] > hw - blob:
                                b[v] = -b[v]
                                b[ax] = min(max(b[ax], 0), hw - blob)
                        boxes.append((b[0], b[1], blob))          # area being covered
                    img[b[0]:b[0] + blob, b[1]:b[1] + blob, :] = b[4]
                if t > 0:
                    hit_all[c * g2:(c + 1) * g2] |= _blob_touch(cfg, boxes)
            if noise_sigma > 0:
                img = img + rng.standard_normal(img.shape, dtype=np.float32) * np.float32(noise_sigma)
            frames[t, c] = np.clip(np.rint(img), 0, 255).astype(np.uint8)
        if t > 0:
            jitter = rng.standard_normal(cur_feat.shape, dtype=np.float32) * np.float32(1e-3)
            fresh = rng.standard_normal(cur_feat.shape, dtype=np.float32)
            cur_feat = np.where(hit_all[:, None], fresh, cur_feat + jitter)
        feats[t] = f32_to_bf16(cur_feat)
        touched.append(np.nonzero(hit_all)[0])
    return Episode(frames=frames, feats=feats, touched=touched)


# --------------------------------------------------------------------------- #
# scripted attention (stand-in for the previous step's text-to-vision scores)
# --------------------------------------------------------------------------- #
def scripted_attention(cfg: ModelConfig, seed: int, hot_tokens: Optional[np.ndarray] = None,
                       uniform: bool = False) -> np.ndarray:
    """fp32 ``[n_layers, n_heads, n_vision]`` rows that are non-negative and sum to < 1.

    With depth the mass concentrates (per-layer sharpness rises, with a partial rebound
    in the last quarter of the layers); ``hot_tokens`` receive extra mass in every layer.
    """
    rng = np.random.default_rng(seed + 15485863)
    lv = cfg.n_vision
    out = np.empty((cfg.n_layers, cfg.n_heads, lv), dtype=np.float32)
    for l in range(cfg.n_layers):
        if uniform:
            out[l] = np.float32(0.5 / lv)
            continue
        depth = l / max(cfg.n_layers - 1, 1)
        sharp = 0.3 + 3.0 * depth - (2.0 * max(depth - 0.75, 0.0)) * 3.0
        for h in range(cfg.n_heads):
            z = rng.standard_normal(lv) * sharp
            if hot_tokens is not None and len(hot_tokens):
                z[hot_tokens] += 2.0 + 2.0 * depth
            w = np.exp(z - z.max())
            out[l, h] = (0.6 * w / w.sum()).astype(np.float32)
    return out
