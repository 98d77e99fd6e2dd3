"""CPU checker for the VLA-Cache control step (arxiv 2502.02175).  TEST INFRASTRUCTURE.

This file is a plain, slow, fp64 restatement of what one control step computes:
token selection (Sec. 3.2-3.4, Algorithm 1), and the partial decoder forward with
per-token K/V reuse (Algorithm 2, Sec. 4.1, Appendix "Inference Detail"), followed by
greedy generation of the action tokens.  It exists only so that tests, the smoke
check and the benchmark's CPU-baseline leg can compare the CUDA library against it;
the library never calls it and shares no code with it.

Conventions
-----------
* Everything is float64 except pixel sums, which are exact integers.
* Model weights arrive as bf16 bit patterns (uint16) and are widened, never rounded.
* By default (``operands="exact"``) the K/V cache, hidden states and attention scores are
  kept in float64 and nothing is rounded.
* The paper runs its models in BF16 (Sec. 5, implementation details; Appendix
  "Experimental Settings").  ``operands="bf16"`` is that precision for the contractions:
  every operand of a matrix product (normalised rows, queries, keys, values, attention
  probabilities, attention output, MLP activations, the row entering the lm_head) is
  rounded to the nearest bf16 value before the product, and keys and values are stored in
  the cache as bf16; sums, the residual stream and everything else stay float64.  The
  distance between the two settings is what bf16 operands cost on a given network; it
  grows with depth (tests/test_oracle_decoder.py measures it).
* Matrix products use ``numpy.matmul``; there is no blocking, fusion or reordering
  beyond what the cited passage states.

Where the paper is silent the reading taken is stated in the function's docstring.

Pins (tests/test_oracle_*.py): closed forms and brute force for the selection
functions; a torch-CPU composition of textbook operators for the dense layer; the
reuse-ratio-0, causality and identical-input identities for the cached step.
Parity with the authors' own code is unpinned: the paper prints no worked numeric
example, so the readings below cannot be checked against their numbers.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------- #
# data carriers
# --------------------------------------------------------------------------- #
def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bf16 value (ties to even), returned as float64.  NaN and inf pass through."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    out = r.view(np.float32).astype(np.float64)
    bad = ~np.isfinite(f)
    if bad.any():
        out[bad] = f[bad]
    return out


def _operand(x: np.ndarray, operands: str) -> np.ndarray:
    if operands == "exact":
        return x
    if operands == "bf16":
        return round_bf16(x)
    raise ValueError(f"operands must be 'exact' or 'bf16', not {operands!r}")


# Optional memo of widened matrices (format conversion only, no arithmetic).  Off by default; tests that
# call the same layer many times switch it on to avoid re-widening hundreds of MB per call.
WIDEN_CACHE_MAX = 0
_widen_cache: Dict[int, tuple] = {}


def _widen_cached(bits: np.ndarray) -> np.ndarray:
    if WIDEN_CACHE_MAX <= 0:
        return widen_bf16(bits)
    key = id(bits)
    hit = _widen_cache.get(key)
    if hit is not None and hit[0] is bits:
        return hit[1]
    if len(_widen_cache) >= WIDEN_CACHE_MAX:
        _widen_cache.clear()
    wide = widen_bf16(bits)
    _widen_cache[key] = (bits, wide)
    return wide


@dataclass
class SelectParams:
    """Hyper-parameters of Algorithm 1 and Eq. (reuse_ratio).

    Appendix "Experimental Settings": tau = 0.996, top-k = 100, tau_task = 0.5.
    ``k_ent`` is the k of Eq. (reuse_ratio); the paper gives no value for it.
    """
    tau: float = 0.996
    top_k: int = 100
    tau_task: float = 0.5
    task_mode: int = 0                      # 0: rank fraction, 1: absolute score test
    k_ent: float = 1.0
    alpha_override: Optional[Sequence[float]] = None
    layer_mask: Optional[Sequence[bool]] = None   # the set of "selected layers" in Sec. 3.3


@dataclass
class Selection:
    sim: np.ndarray                  # [L_v] float64
    static_mask: np.ndarray          # [L_v] bool
    S_layer: np.ndarray              # [n_layers, L_v]
    S: np.ndarray                    # [L_v]
    task_mask: np.ndarray
    final_mask: np.ndarray
    entropy: np.ndarray              # [n_layers + 1], entry 0 is the reference entropy
    ratio: np.ndarray                # [n_layers]   R^l
    alpha: np.ndarray                # [n_layers]   Eq. (reuse_ratio), clamped to [0, 1]
    alpha_bar: np.ndarray            # [n_layers]   running maximum of alpha
    n_reuse: np.ndarray              # [n_layers]   int
    reuse_order: np.ndarray          # P_final ordered least task-relevant first (token ids)
    rows: List[np.ndarray]           # per layer: ascending positions to recompute
    M: np.ndarray                    # [n_layers] int, len(rows[l])


@dataclass
class CacheState:
    """What persists between control steps for one sequence."""
    K: np.ndarray                    # [n_layers, max_seq, n_heads, head_dim]
    V: np.ndarray
    prev_frames: Optional[np.ndarray] = None     # uint8 [n_cams, H, W, 3]
    attn_tv: Optional[np.ndarray] = None         # [n_layers, n_heads, L_v]
    warm: bool = False


def new_cache(cfg) -> CacheState:
    shape = (cfg.n_layers, cfg.max_seq, cfg.n_heads, cfg.head_dim)
    return CacheState(K=np.zeros(shape), V=np.zeros(shape))


# --------------------------------------------------------------------------- #
# Sec. 3.2  static token selection
# --------------------------------------------------------------------------- #
def patch_similarity(frames_t: np.ndarray, frames_prev: np.ndarray, grid: int, patch: int) -> np.ndarray:
    """Eq. (sim): cosine similarity of each raw pixel patch with the same patch one frame earlier.

    ``frames_*`` are uint8 ``[n_cams, H, W, 3]``.  A patch is the ``patch x patch x 3`` block
    flattened to one vector of raw 0..255 values (no centring).  Token ``cam*grid*grid +
    i*grid + j`` is the patch in block-row ``i``, block-column ``j`` of camera ``cam``.
    Sums are exact integers; one sqrt and one divide in float64 follow.
    Reading for 0/0: two all-zero patches are identical (1.0); one all-zero patch gives 0.0.
    """
    n_cams = frames_t.shape[0]
    sim = np.empty(n_cams * grid * grid, dtype=np.float64)
    for cam in range(n_cams):
        for i in range(grid):
            for j in range(grid):
                a = frames_t[cam, i * patch:(i + 1) * patch, j * patch:(j + 1) * patch, :].astype(np.int64).reshape(-1)
                b = frames_prev[cam, i * patch:(i + 1) * patch, j * patch:(j + 1) * patch, :].astype(np.int64).reshape(-1)
                dot, na, nb = int(np.sum(a * b)), int(np.sum(a * a)), int(np.sum(b * b))
                if na == 0 and nb == 0:
                    s = 1.0
                elif na == 0 or nb == 0:
                    s = 0.0
                else:
                    s = float(np.float64(dot) / np.sqrt(np.float64(na * nb)))
                sim[cam * grid * grid + i * grid + j] = s
    return sim


def patch_similarity_values(frames_t: np.ndarray, frames_prev: np.ndarray, grid: int, patch: int) -> np.ndarray:
    """Eq. (sim) on frames given as real values ``[n_cams, H, W, 3]`` (normalised pixels rather than raw bytes; the
    Appendix's noisy real-robot setting): the same patch layout and 0/0 readings as ``patch_similarity``, sums in
    float64.  Values may be negative, so the similarity ranges over [-1, 1]."""
    ft = np.asarray(frames_t, dtype=np.float64)
    fp = np.asarray(frames_prev, dtype=np.float64)
    n_cams = ft.shape[0]
    sim = np.empty(n_cams * grid * grid, dtype=np.float64)
    for cam in range(n_cams):
        for i in range(grid):
            for j in range(grid):
                a = ft[cam, i * patch:(i + 1) * patch, j * patch:(j + 1) * patch, :].reshape(-1)
                b = fp[cam, i * patch:(i + 1) * patch, j * patch:(j + 1) * patch, :].reshape(-1)
                dot, na, nb = math.fsum(a * b), math.fsum(a * a), math.fsum(b * b)
                if na == 0.0 and nb == 0.0:
                    s = 1.0
                elif na == 0.0 or nb == 0.0:
                    s = 0.0
                else:
                    s = dot / math.sqrt(na * nb)
                sim[cam * grid * grid + i * grid + j] = s
    return sim


def static_tokens(sim: np.ndarray, tau: float, top_k: int) -> np.ndarray:
    """Eq. (topk): of the tokens with ``sim >= tau`` keep the ``top_k`` most similar.

    Reading: the threshold is inclusive; equal similarities rank the lower index first;
    if fewer than ``top_k`` tokens pass the threshold all of them are kept.
    """
    cand = [v for v in range(len(sim)) if sim[v] >= tau]
    cand.sort(key=lambda v: (-sim[v], v))
    mask = np.zeros(len(sim), dtype=bool)
    for v in cand[:max(top_k, 0)]:
        mask[v] = True
    return mask


# --------------------------------------------------------------------------- #
# Sec. 3.3  task relevance
# --------------------------------------------------------------------------- #
def task_relevance(attn_tv: np.ndarray, layer_mask: Optional[Sequence[bool]] = None):
    """Eq. (avistext) and the two means after it.

    ``attn_tv[l, h, v]`` is the attention probability that head ``h`` of layer ``l`` put on
    vision key ``v``, already averaged over the prompt-text query rows that follow the vision
    block (the text-to-vision block of the attention tensor).  ``S_layer[l] = Mean_heads``,
    ``S = Mean over the selected layers``.  Sums run in index order in float64.
    """
    n_layers, n_heads, lv = attn_tv.shape
    S_layer = np.zeros((n_layers, lv), dtype=np.float64)
    for l in range(n_layers):
        acc = np.zeros(lv, dtype=np.float64)
        for h in range(n_heads):
            acc = acc + attn_tv[l, h].astype(np.float64)
        S_layer[l] = acc / np.float64(n_heads)
    chosen = [l for l in range(n_layers) if layer_mask is None or layer_mask[l]]
    acc = np.zeros(lv, dtype=np.float64)
    for l in chosen:
        acc = acc + S_layer[l]
    S = acc / np.float64(max(len(chosen), 1))
    return S_layer, S


def task_relevant_tokens(S: np.ndarray, tau_task: float, task_mode: int = 0) -> np.ndarray:
    """Eq. (ptask).

    ``task_mode = 1`` is the printed test ``S >= tau_task``.  ``task_mode = 0`` (default
    reading) treats tau_task as a rank fraction: the vision tokens are ranked by S (higher
    first, ties to the lower index) and the top ``L_v - floor(tau_task * L_v)`` are
    task-relevant.  Attention probabilities over L_v tokens sum to at most 1, so the
    printed absolute test with tau_task = 0.5 could never select anything.
    """
    lv = len(S)
    mask = np.zeros(lv, dtype=bool)
    if task_mode == 1:
        for v in range(lv):
            mask[v] = S[v] >= tau_task
        return mask
    n_task = lv - int(math.floor(tau_task * lv))
    n_task = min(max(n_task, 0), lv)
    order = sorted(range(lv), key=lambda v: (-S[v], v))
    for v in order[:n_task]:
        mask[v] = True
    return mask


def reusable_tokens(static_mask: np.ndarray, task_mask: np.ndarray) -> np.ndarray:
    """Eq. (pfinal): static tokens that are not task-relevant."""
    return static_mask & ~task_mask


# --------------------------------------------------------------------------- #
# Sec. 3.4  layer-adaptive reuse
# --------------------------------------------------------------------------- #
def attention_entropy(S_l: np.ndarray) -> float:
    """Entropy (natural log) of the head-and-text-mean attention of one layer over the
    vision tokens, renormalised to sum to one; 0 ln 0 = 0.  An all-zero row is read as
    the uniform distribution."""
    total = 0.0
    for x in S_l:
        total += float(x)
    if total <= 0.0:
        return math.log(len(S_l))
    e = 0.0
    for x in S_l:
        p = float(x) / total
        if p > 0.0:
            e -= p * math.log(p)
    return e


def reuse_ratios(S_layer: np.ndarray, k_ent: float):
    """Sec. 3.4: ``R^l = (E^{l-1} - E^l) / E^{l-1}`` and Eq. (reuse_ratio)
    ``alpha^l = min(k * sum_{j<=l} R^j, 1)``.

    Readings: the entropy before the first layer is that of the uniform distribution,
    ``ln L_v``; a zero ``E^{l-1}`` gives ``R^l = 0``; negative cumulative sums clamp to 0.
    ``alpha_bar`` is the running maximum over depth: a token skipped in one layer has no
    hidden state to resume from, so the reuse sets must be nested.
    """
    n_layers, lv = S_layer.shape
    E = np.empty(n_layers + 1, dtype=np.float64)
    E[0] = math.log(lv)
    for l in range(n_layers):
        E[l + 1] = attention_entropy(S_layer[l])
    R = np.zeros(n_layers, dtype=np.float64)
    alpha = np.zeros(n_layers, dtype=np.float64)
    alpha_bar = np.zeros(n_layers, dtype=np.float64)
    cum, run = 0.0, 0.0
    for l in range(n_layers):
        R[l] = (E[l] - E[l + 1]) / E[l] if E[l] > 0.0 else 0.0
        cum += R[l]
        alpha[l] = min(max(k_ent * cum, 0.0), 1.0)
        run = max(run, alpha[l])
        alpha_bar[l] = run
    return E, R, alpha, alpha_bar


def reuse_order(final_mask: np.ndarray, S: np.ndarray) -> np.ndarray:
    """P_final ordered least task-relevant first (ascending S, ties to the lower index):
    the tokens that matter most for the task are the last to be reused."""
    ids = [v for v in range(len(final_mask)) if final_mask[v]]
    ids.sort(key=lambda v: (S[v], v))
    return np.asarray(ids, dtype=np.int64)


def select(cfg, frames_t: np.ndarray, cache: CacheState, params: SelectParams,
           force_full: bool = False, frame_values: bool = False) -> Selection:
    """Algorithm 1 followed by line 3 of Algorithm 2: which positions each layer recomputes.

    Layer ``l`` reuses the first ``floor(alpha_bar^l * |P_final|)`` tokens of ``reuse_order``;
    every text position and every other vision position is recomputed.  On a cold cache
    (no previous frame) nothing is reusable.
    """
    lv, L, nl = cfg.n_vision, cfg.seq_len, cfg.n_layers
    all_rows = np.arange(L, dtype=np.int64)
    if force_full or not cache.warm:
        z = np.zeros(lv, dtype=bool)
        return Selection(sim=np.zeros(lv), static_mask=z, S_layer=np.zeros((nl, lv)), S=np.zeros(lv),
                         task_mask=z.copy(), final_mask=z.copy(), entropy=np.zeros(nl + 1),
                         ratio=np.zeros(nl), alpha=np.zeros(nl), alpha_bar=np.zeros(nl),
                         n_reuse=np.zeros(nl, dtype=np.int64), reuse_order=np.zeros(0, dtype=np.int64),
                         rows=[all_rows.copy() for _ in range(nl)], M=np.full(nl, L, dtype=np.int64))
    if frame_values:      # frames and cache.prev_frames hold real values (normalised pixels), not bytes
        sim = patch_similarity_values(frames_t, cache.prev_frames, cfg.grid, cfg.patch)
    else:
        sim = patch_similarity(frames_t, cache.prev_frames, cfg.grid, cfg.patch)
    static_mask = static_tokens(sim, params.tau, params.top_k)
    S_layer, S = task_relevance(cache.attn_tv, params.layer_mask)
    task_mask = task_relevant_tokens(S, params.tau_task, params.task_mode)
    final_mask = reusable_tokens(static_mask, task_mask)
    E, R, alpha, alpha_bar = reuse_ratios(S_layer, params.k_ent)
    if params.alpha_override is not None:
        run = 0.0
        for l in range(nl):
            run = max(run, min(max(float(params.alpha_override[l]), 0.0), 1.0))
            alpha_bar[l] = run
    order = reuse_order(final_mask, S)
    n_final = len(order)
    n_reuse = np.zeros(nl, dtype=np.int64)
    rows: List[np.ndarray] = []
    for l in range(nl):
        n_reuse[l] = int(math.floor(alpha_bar[l] * n_final))
        skipped = np.zeros(L, dtype=bool)
        for v in order[:n_reuse[l]]:
            skipped[cfg.n_text_pre + int(v)] = True
        rows.append(all_rows[~skipped])
    return Selection(sim=sim, static_mask=static_mask, S_layer=S_layer, S=S, task_mask=task_mask,
                     final_mask=final_mask, entropy=E, ratio=R, alpha=alpha, alpha_bar=alpha_bar,
                     n_reuse=n_reuse, reuse_order=order, rows=rows,
                     M=np.asarray([len(r) for r in rows], dtype=np.int64))


# --------------------------------------------------------------------------- #
# decoder layer (Llama-2 shape: RMSNorm, rotary attention, SwiGLU, no biases)
# --------------------------------------------------------------------------- #
def rms_norm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x * gain / sqrt(mean(x^2) + eps), row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, positions: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotary embedding, rotate-half pairing: element ``i`` pairs with ``i + d/2``.

    ``x`` is ``[rows, heads, d]``; row ``r`` is rotated by the angles of ``positions[r]``
    (Appendix "Rotary Embedding": recomputed tokens get the rotation of their own,
    unchanged, position).  ``cos``/``sin`` are ``[max_seq, d/2]`` tables.
    """
    half = x.shape[-1] // 2
    c = cos[positions].astype(np.float64)[:, None, :]
    s = sin[positions].astype(np.float64)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def layer_forward(cfg, layer_w: Dict[str, np.ndarray], K: np.ndarray, V: np.ndarray,
                  hidden: np.ndarray, rows: np.ndarray, cos: np.ndarray, sin: np.ndarray,
                  emit_attention: bool = True, block_start: Optional[int] = None,
                  operands: str = "exact", hidden_keys: Optional[np.ndarray] = None) -> Optional[np.ndarray]:
    """One decoder layer over the positions in ``rows`` only (Algorithm 2, Sec. 4.1).

    ``K``/``V`` are this layer's cache ``[max_seq, heads, d]`` and are updated in place at
    ``rows``; every other position keeps the entry written in an earlier step.  ``hidden``
    is ``[>= max(rows)+1, hidden]`` and is updated in place at ``rows``.  A recomputed query
    at position ``p`` attends to all cache positions ``<= p`` (Sec. 3.1 attention; the mask
    follows original positions, Appendix "Position and Attention Masking"), whether their
    K/V are fresh or reused.  Keys are stored after rotation.  With ``block_start`` the rows
    at positions ``>= block_start`` form one block that is decoded in parallel: each of them
    also sees the block's later positions (see ``step_chunk``).

    ``hidden_keys`` (bool ``[max_seq]``) marks cache positions no query may attend to (tokens
    removed from the sequence by ``step_pruned``).

    ``operands="bf16"`` rounds every operand of a matrix product to bf16 first and stores keys and values
    as bf16 (the paper's BF16 setting; see the module header); the emitted probabilities are not rounded.

    Returns, if asked, ``[heads, L_v]``: the softmax probability on each vision key averaged
    over the prompt-text query rows that follow the vision block (Eq. avistext, read as
    text queries x vision keys).
    """
    H, d = cfg.n_heads, cfg.head_dim
    rows = np.asarray(rows, dtype=np.int64)
    W = {k: _widen_cached(v) for k, v in layer_w.items()}
    x = hidden[rows]
    xn = _operand(rms_norm(x, W["g_attn"], cfg.rms_eps), operands)
    q = (xn @ W["wq"].T).reshape(len(rows), H, d)
    k = (xn @ W["wk"].T).reshape(len(rows), H, d)
    v = (xn @ W["wv"].T).reshape(len(rows), H, d)
    q = _operand(rope(q, rows, cos, sin), operands)
    k = rope(k, rows, cos, sin)
    K[rows] = _operand(k, operands)
    V[rows] = _operand(v, operands)

    n_keys = int(rows.max()) + 1
    key_pos = np.arange(n_keys)
    visible = key_pos[None, :] <= rows[:, None]                      # [rows, keys]
    if block_start is not None:
        visible = visible | ((rows[:, None] >= block_start) & (key_pos[None, :] >= block_start))
    if hidden_keys is not None:
        visible = visible & ~np.asarray(hidden_keys, dtype=bool)[None, :n_keys]
    v0 = cfg.n_text_pre
    v1 = v0 + cfg.n_vision
    text_q = (rows >= v1) & (rows < cfg.seq_len)
    attn_out = np.empty((len(rows), H, d), dtype=np.float64)
    emitted = np.zeros((H, cfg.n_vision), dtype=np.float64)
    for h in range(H):
        scores = (q[:, h, :] @ K[:n_keys, h, :].T) / math.sqrt(d)
        scores = np.where(visible, scores, -np.inf)
        scores = scores - scores.max(axis=1, keepdims=True)
        p = np.exp(scores)
        p = p / p.sum(axis=1, keepdims=True)
        attn_out[:, h, :] = _operand(p, operands) @ V[:n_keys, h, :]
        if emit_attention and text_q.any():
            emitted[h] = p[text_q][:, v0:v1].mean(axis=0)
    x = x + _operand(attn_out.reshape(len(rows), H * d), operands) @ W["wo"].T
    xn = _operand(rms_norm(x, W["g_mlp"], cfg.rms_eps), operands)
    x = x + _operand(silu(xn @ W["w_gate"].T) * (xn @ W["w_up"].T), operands) @ W["w_down"].T
    hidden[rows] = x
    return emitted if emit_attention else None


# --------------------------------------------------------------------------- #
# one control step
# --------------------------------------------------------------------------- #
@dataclass
class StepResult:
    tokens: np.ndarray               # [n_action] this checker's own greedy choices
    fed_tokens: np.ndarray           # [n_action] tokens actually fed back (forced or own)
    logits: np.ndarray               # [n_action, vocab]
    margins: np.ndarray              # [n_action] top-1 minus top-2 logit
    selection: Selection
    hidden: np.ndarray               # [max_seq, hidden] after the last layer
    attn_tv: np.ndarray              # [n_layers, heads, L_v] emitted by this step's prefill


def input_rows(cfg, model: Dict[str, object], feats_bf16: np.ndarray, prompt_ids: np.ndarray,
               rows0: Optional[np.ndarray] = None) -> np.ndarray:
    """Hidden rows entering layer 0: token embeddings at the text positions, projected
    vision features (one linear map) at the vision positions.

    With ``rows0`` (the positions layer 0 recomputes) only those vision positions are
    projected (Sec. 4.1: ``H_t`` is needed for the tokens that are not reused); the other
    vision rows stay zero.  The reuse sets are nested over depth, so a row that layer 0
    skips is read by no layer."""
    hidden = np.zeros((cfg.max_seq, cfg.hidden), dtype=np.float64)
    embed = model["embed"]
    v0, v1 = cfg.n_text_pre, cfg.n_text_pre + cfg.n_vision
    ids = np.asarray(prompt_ids, dtype=np.int64)
    hidden[:v0] = widen_bf16(embed[ids[:v0]])
    hidden[v1:cfg.seq_len] = widen_bf16(embed[ids[v0:]])
    if rows0 is None:
        hidden[v0:v1] = widen_bf16(feats_bf16) @ widen_bf16(model["proj"]).T
    else:
        vis = np.asarray([p for p in np.asarray(rows0, dtype=np.int64) if v0 <= p < v1], dtype=np.int64)
        if len(vis):
            hidden[vis] = widen_bf16(np.asarray(feats_bf16)[vis - v0]) @ widen_bf16(model["proj"]).T
    return hidden


def _logits(cfg, model, h_row: np.ndarray, operands: str = "exact") -> np.ndarray:
    xn = _operand(rms_norm(h_row[None, :], widen_bf16(model["g_final"]), cfg.rms_eps), operands)
    return (xn @ _widen_cached(model["lm_head"]).T)[0]


def step(cfg, model: Dict[str, object], cache: CacheState, frames_t: np.ndarray,
         feats_bf16: np.ndarray, prompt_ids: np.ndarray, params: SelectParams,
         force_full: bool = False, forced_tokens: Optional[Sequence[int]] = None,
         selection: Optional[Selection] = None, operands: str = "exact") -> StepResult:
    """Selection, partial prefill, then greedy decoding of ``n_action`` tokens.

    The first action token is the argmax (ties to the lower id) of the logits at the last
    prefill position; each further token comes from one ordinary single-row pass that
    appends its K/V behind the prefill (Sec. 3.1 cache append; the paper generates 7 action
    tokens and notes that tokens after the first cost the same with or without reuse).
    The appended entries are overwritten by the next step.  ``forced_tokens`` replaces the
    fed-back tokens (used when a comparison run must follow another implementation's
    choices); this checker's own choices are still reported.
    """
    sel = selection if selection is not None else select(cfg, frames_t, cache, params, force_full)
    cos, sin = model["rope_cos"], model["rope_sin"]
    hidden = input_rows(cfg, model, feats_bf16, prompt_ids, rows0=sel.rows[0])
    attn_next = np.zeros((cfg.n_layers, cfg.n_heads, cfg.n_vision), dtype=np.float64)
    for l in range(cfg.n_layers):
        attn_next[l] = layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden,
                                     sel.rows[l], cos, sin, emit_attention=True, operands=operands)
    L = cfg.seq_len
    tokens = np.zeros(cfg.n_action, dtype=np.int64)
    fed = np.zeros(cfg.n_action, dtype=np.int64)
    logits = np.zeros((cfg.n_action, cfg.vocab), dtype=np.float64)
    margins = np.zeros(cfg.n_action, dtype=np.float64)
    for i in range(cfg.n_action):
        pos = L - 1 + i
        if i > 0:
            hidden[pos] = widen_bf16(model["embed"][int(fed[i - 1])])
            for l in range(cfg.n_layers):
                layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden,
                              np.asarray([pos]), cos, sin, emit_attention=False, operands=operands)
        logits[i] = _logits(cfg, model, hidden[pos], operands)
        tokens[i] = int(np.argmax(logits[i]))
        top2 = np.partition(logits[i], -2)[-2:]
        margins[i] = float(top2[1] - top2[0])
        fed[i] = tokens[i] if forced_tokens is None else int(forced_tokens[i])
    cache.attn_tv = attn_next
    cache.prev_frames = np.array(frames_t, copy=True)
    cache.warm = True
    return StepResult(tokens=tokens, fed_tokens=fed, logits=logits, margins=margins,
                      selection=sel, hidden=hidden, attn_tv=attn_next)


def step_chunk(cfg, model: Dict[str, object], cache: CacheState, frames_t: np.ndarray,
               feats_bf16: np.ndarray, prompt_ids: np.ndarray, params: SelectParams,
               act_embed_bf16: np.ndarray, force_full: bool = False,
               selection: Optional[Selection] = None, operands: str = "exact") -> StepResult:
    """Selection and partial prefill as in ``step``, then ALL action tokens from one pass.

    The paper applies the method unchanged to OpenVLA-OFT, whose decoder emits its action
    chunk in one pass (Sec. 5, main LIBERO results, Table 2), and gives no equations for that
    decoder.  Reading taken
    here: behind the prompt sit ``n_action`` placeholder rows at positions ``L .. L+n_action-1``
    whose input is the fixed embedding ``act_embed_bf16[i]`` (a weight, not a fed-back token).
    They run through every layer together: each sees the whole prompt (reused or fresh K/V, as
    the prefill left it) and every row of the chunk, in both directions; their K/V are written
    behind the prompt and overwritten by the next step.  Token ``i`` is the argmax (ties to the
    lower id) of the logits of row ``L+i``.  The prefill's own last-row logits are not used.
    ``fed_tokens`` of the result equals ``tokens``: nothing is fed back.
    """
    sel = selection if selection is not None else select(cfg, frames_t, cache, params, force_full)
    cos, sin = model["rope_cos"], model["rope_sin"]
    hidden = input_rows(cfg, model, feats_bf16, prompt_ids, rows0=sel.rows[0])
    attn_next = np.zeros((cfg.n_layers, cfg.n_heads, cfg.n_vision), dtype=np.float64)
    for l in range(cfg.n_layers):
        attn_next[l] = layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden,
                                     sel.rows[l], cos, sin, emit_attention=True, operands=operands)
    L, n = cfg.seq_len, cfg.n_action
    chunk_rows = np.arange(L, L + n, dtype=np.int64)
    hidden[chunk_rows] = widen_bf16(np.asarray(act_embed_bf16).reshape(n, cfg.hidden))
    for l in range(cfg.n_layers):
        layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden, chunk_rows, cos, sin,
                      emit_attention=False, block_start=L, operands=operands)
    tokens = np.zeros(n, dtype=np.int64)
    logits = np.zeros((n, cfg.vocab), dtype=np.float64)
    margins = np.zeros(n, dtype=np.float64)
    for i in range(n):
        logits[i] = _logits(cfg, model, hidden[L + i], operands)
        tokens[i] = int(np.argmax(logits[i]))
        top2 = np.partition(logits[i], -2)[-2:]
        margins[i] = float(top2[1] - top2[0])
    cache.attn_tv = attn_next
    cache.prev_frames = np.array(frames_t, copy=True)
    cache.warm = True
    return StepResult(tokens=tokens, fed_tokens=tokens.copy(), logits=logits, margins=margins,
                      selection=sel, hidden=hidden, attn_tv=attn_next)


# --------------------------------------------------------------------------- #
# comparison baseline: intra-frame pruning after layer K (FastV-style)
# --------------------------------------------------------------------------- #
def pruned_vision_tokens(score: np.ndarray, n_keep: int) -> np.ndarray:
    """The ``n_keep`` vision tokens with the highest score (ties to the lower index) as a bool mask."""
    order = sorted(range(len(score)), key=lambda v: (-score[v], v))
    keep = np.zeros(len(score), dtype=bool)
    for v in order[:max(min(n_keep, len(score)), 0)]:
        keep[v] = True
    return keep


def step_pruned(cfg, model: Dict[str, object], cache: CacheState, frames_t: np.ndarray,
                feats_bf16: np.ndarray, prompt_ids: np.ndarray, prune_layer: int, n_keep: int,
                forced_tokens: Optional[Sequence[int]] = None, operands: str = "exact",
                prune_scores: Optional[np.ndarray] = None) -> StepResult:
    """The baseline the paper compares with in its main LIBERO table (row "+FastV"; Sec. 5, baselines): no reuse
    across frames; instead, inside one frame, vision tokens that receive little attention are dropped part-way
    through the decoder.  The paper gives no equations for it; reading taken here (that of the FastV method):

    * layers ``0 .. prune_layer-1`` run over the whole sequence;
    * every vision token gets the score ``mean over heads and over the prompt-text query rows behind the vision
      block`` of the attention probability it received in layer ``prune_layer-1`` (the text-to-vision scores of
      Eq. (avistext) that every prefill emits); the ``n_keep`` best are kept, ties to the lower index;
    * from layer ``prune_layer`` on, the dropped tokens are gone: their rows are not computed and no query attends
      to their positions, in the prefill and in the single-row passes of the action tokens; kept tokens and text
      keep their original positions (and so their rotary angles).

    ``prune_scores`` (``[heads, L_v]``) replaces this run's own layer ``prune_layer-1`` scores in the ranking (a
    replayed comparison ranks by another implementation's scores so that the kept sets can be compared exactly).
    ``prune_layer >= n_layers`` or ``n_keep >= L_v`` is the plain full step.  The cache is used as scratch for this
    step's K/V and is left warm like after ``step`` (previous frame, emitted scores); ``selection.M`` reports the
    rows per layer.
    """
    nl, L, lv = cfg.n_layers, cfg.seq_len, cfg.n_vision
    sel = select(cfg, frames_t, cache, SelectParams(), force_full=True)
    cos, sin = model["rope_cos"], model["rope_sin"]
    hidden = input_rows(cfg, model, feats_bf16, prompt_ids)
    attn_next = np.zeros((nl, cfg.n_heads, lv), dtype=np.float64)
    hidden_keys = None
    rows = np.arange(L, dtype=np.int64)
    v0 = cfg.n_text_pre
    kept = np.ones(lv, dtype=bool)
    for l in range(nl):
        if l == prune_layer and l > 0 and n_keep < lv:
            score = np.zeros(lv, dtype=np.float64)
            src = attn_next[l - 1] if prune_scores is None else np.asarray(prune_scores, dtype=np.float64)
            for h in range(cfg.n_heads):
                score = score + src[h]
            kept = pruned_vision_tokens(score / np.float64(cfg.n_heads), n_keep)
            hidden_keys = np.zeros(cfg.max_seq, dtype=bool)
            hidden_keys[v0:v0 + lv] = ~kept
            rows = np.asarray([p for p in range(L) if not hidden_keys[p]], dtype=np.int64)
        sel.rows[l], sel.M[l] = rows, len(rows)
        attn_next[l] = layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden, rows, cos, sin,
                                     emit_attention=True, operands=operands, hidden_keys=hidden_keys)
    tokens = np.zeros(cfg.n_action, dtype=np.int64)
    fed = np.zeros(cfg.n_action, dtype=np.int64)
    logits = np.zeros((cfg.n_action, cfg.vocab), dtype=np.float64)
    margins = np.zeros(cfg.n_action, dtype=np.float64)
    for i in range(cfg.n_action):
        pos = L - 1 + i
        if i > 0:
            hidden[pos] = widen_bf16(model["embed"][int(fed[i - 1])])
            for l in range(nl):
                hk = hidden_keys if (hidden_keys is not None and l >= prune_layer) else None
                layer_forward(cfg, model["layers"][l], cache.K[l], cache.V[l], hidden, np.asarray([pos]), cos, sin,
                              emit_attention=False, operands=operands, hidden_keys=hk)
        logits[i] = _logits(cfg, model, hidden[pos], operands)
        tokens[i] = int(np.argmax(logits[i]))
        top2 = np.partition(logits[i], -2)[-2:]
        margins[i] = float(top2[1] - top2[0])
        fed[i] = tokens[i] if forced_tokens is None else int(forced_tokens[i])
    cache.attn_tv = attn_next
    cache.prev_frames = np.array(frames_t, copy=True)
    cache.warm = True
    sel.final_mask = ~kept                    # reported for inspection: the dropped vision tokens
    return StepResult(tokens=tokens, fed_tokens=fed, logits=logits, margins=margins,
                      selection=sel, hidden=hidden, attn_tv=attn_next)
