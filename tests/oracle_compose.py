"""Compositions of the CPU checker's own functions used by the tests (no arithmetic of their own).

``step_layer_major`` runs one control step with the loops interchanged: every layer is taken once and
sees first the prefill rows, then the single rows of the action tokens one after the other.  With the
fed-back tokens known in advance (a replayed comparison feeds the library's tokens) the input of every
single-row pass is known before any layer runs, layer ``l`` of row ``i`` needs only layer ``l - 1`` of the
same row and layer ``l``'s cache rows of earlier positions, so the result is the one ``oracle.step``
gives (``tests/test_oracle_decoder.py`` checks that they are bit-identical).  What it buys: a layer's
weights are widened to float64 once per step instead of once per pass, which is what makes a 32-layer
7B-shaped step affordable inside a test.
"""
from __future__ import annotations

import numpy as np

from oracle import vla_cache_oracle as orc


def step_layer_major(cfg, model, cache, frames_t, feats_bf16, prompt_ids, params, forced_tokens,
                     force_full=False, selection=None, operands="exact") -> orc.StepResult:
    sel = selection if selection is not None else orc.select(cfg, frames_t, cache, params, force_full)
    cos, sin = model["rope_cos"], model["rope_sin"]
    hidden = orc.input_rows(cfg, model, feats_bf16, prompt_ids, rows0=sel.rows[0])
    L, n = cfg.seq_len, cfg.n_action
    fed = np.asarray(forced_tokens, dtype=np.int64).reshape(n)
    for i in range(1, n):
        hidden[L - 1 + i] = orc.widen_bf16(model["embed"][int(fed[i - 1])])
    attn_next = np.zeros((cfg.n_layers, cfg.n_heads, cfg.n_vision), dtype=np.float64)
    for l in range(cfg.n_layers):
        lw, K, V = model["layers"][l], cache.K[l], cache.V[l]
        attn_next[l] = orc.layer_forward(cfg, lw, K, V, hidden, sel.rows[l], cos, sin, emit_attention=True, operands=operands)
        for i in range(1, n):
            orc.layer_forward(cfg, lw, K, V, hidden, np.asarray([L - 1 + i]), cos, sin, emit_attention=False, operands=operands)
    tokens = np.zeros(n, dtype=np.int64)
    logits = np.zeros((n, cfg.vocab), dtype=np.float64)
    margins = np.zeros(n, dtype=np.float64)
    for i in range(n):
        logits[i] = orc._logits(cfg, model, hidden[L - 1 + i], operands)
        tokens[i] = int(np.argmax(logits[i]))
        top2 = np.partition(logits[i], -2)[-2:]
        margins[i] = float(top2[1] - top2[0])
    cache.attn_tv = attn_next
    cache.prev_frames = np.array(frames_t, copy=True)
    cache.warm = True
    return orc.StepResult(tokens=tokens, fed_tokens=fed, logits=logits, margins=margins, selection=sel,
                          hidden=hidden, attn_tv=attn_next)
