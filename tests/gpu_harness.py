"""Shared helpers for the GPU parity tests: run the CUDA library and the CPU checker on the same
seeded inputs and compare them.

Index sets must agree bit for bit; floating-point outputs within ``TOL`` = 2e-2 of the largest
reference magnitude, against the checker in exact arithmetic (``OPERANDS`` = "exact").  That bound holds
for the shallow models of most tests.  Through 32 layers two computations that both round their
matrix-product operands to bf16 drift apart by more than 2e-2, however faithful each is (a difference
far below one bf16 unit in a value that is about to be rounded moves the result by a whole unit with
the matching probability, so differences do not stay small); the 32-layer test therefore measures, on
the CPU alone, how far the checker's own bf16-operand setting is from its exact setting and scales its
tolerance by that figure.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import vla_cache_oracle as orc
from paper_2502_02175_b200 import binding as vb
from paper_2502_02175_b200 import synth

TOL = 2e-2
OPERANDS = "exact"


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |got - ref| / max |ref|."""
    ref = np.asarray(ref, dtype=np.float64)
    denom = float(np.max(np.abs(ref)))
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - ref))) / (denom if denom > 0 else 1.0)


def bf16_tensor_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


class Session:
    """One context + cache of the CUDA library next to one checker state per sequence."""

    def __init__(self, cfg, model, batch=1, dev_model=None):
        self.cfg, self.model, self.batch = cfg, model, batch
        self.dev = dev_model if dev_model is not None else vb.DeviceModel(model)
        self.ctx = vb.vlac_create(vb.make_config(cfg, max_batch=batch), self.dev.weights)
        self.cache = vb.vlac_cache_alloc(self.ctx, batch)
        self.ocache = [orc.new_cache(cfg) for _ in range(batch)]
        self.stream = torch.cuda.Stream()      # a non-default stream: vlac_step replays its CUDA graph there

    def close(self):
        vb.vlac_cache_free(self.cache)
        vb.vlac_destroy(self.ctx)

    # ---- cache access
    def read_attn(self, part, seq=0) -> np.ndarray:
        cfg = self.cfg
        t = torch.empty((cfg.n_layers, cfg.n_heads, cfg.n_vision), dtype=torch.float32, device="cuda")
        vb.vlac_cache_read(self.cache, part, seq, 0, t)
        torch.cuda.synchronize()
        return t.cpu().numpy()

    def read_kv(self, part, layer, seq=0) -> np.ndarray:
        cfg = self.cfg
        t = torch.empty((cfg.max_seq, cfg.n_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
        vb.vlac_cache_read(self.cache, part, seq, layer, t)
        torch.cuda.synchronize()
        return bf16_tensor_to_f64(t)

    def write_kv(self, part, layer, values_f64: np.ndarray, seq=0):
        t = torch.from_numpy(values_f64.astype(np.float32)).to("cuda").to(torch.bfloat16).contiguous()
        vb.vlac_cache_write(self.cache, part, seq, layer, t)

    def set_warm_state(self, prev_frames: np.ndarray, attn: np.ndarray, seq=0):
        """Make sequence ``seq`` warm with the given previous frame and saved attention, on both sides."""
        vb.vlac_cache_write(self.cache, vb.PART_PREV_FRAME, seq, 0, torch.from_numpy(prev_frames).to("cuda").contiguous())
        vb.vlac_cache_write(self.cache, vb.PART_ATTN_PREV, seq, 0, torch.from_numpy(attn.astype(np.float32)).to("cuda").contiguous())
        vb.vlac_cache_write(self.cache, vb.PART_WARM, seq, 0, torch.ones(1, dtype=torch.int32, device="cuda"))
        oc = self.ocache[seq]
        oc.prev_frames, oc.attn_tv, oc.warm = prev_frames.copy(), attn.astype(np.float32).astype(np.float64), True


def oparams(**kw) -> orc.SelectParams:
    return orc.SelectParams(**kw)


def gparams(p: orc.SelectParams):
    mask = 0
    if p.layer_mask is not None:
        for l, on in enumerate(p.layer_mask):
            mask |= (1 << l) if on else 0
    return vb.make_params(p.tau, p.top_k, p.tau_task, p.task_mode, p.k_ent, p.alpha_override, mask)


def check_selection(got: dict, sel: orc.Selection, seq: int, cfg, where=""):
    """Bit-exact comparison of everything that is an index or an exactly defined value."""
    assert np.array_equal(got["sim"][seq], sel.sim), f"{where}: similarity differs"
    assert np.array_equal(got["static_mask"][seq].astype(bool), sel.static_mask), f"{where}: P_static"
    assert np.array_equal(got["S"][seq], sel.S), f"{where}: task-relevance scores differ"
    assert np.array_equal(got["task_mask"][seq].astype(bool), sel.task_mask), f"{where}: P_task"
    assert np.array_equal(got["final_mask"][seq].astype(bool), sel.final_mask), f"{where}: P_final"
    np.testing.assert_allclose(got["alpha"][seq], sel.alpha_bar, atol=1e-11, err_msg=f"{where}: alpha")
    n_final = int(sel.final_mask.sum())
    for l in range(cfg.n_layers):
        x = sel.alpha_bar[l] * n_final
        assert abs(x - round(x)) >= 1e-6 or x == round(x), f"{where}: reuse count of layer {l} sits on a rounding edge"
        m = int(sel.M[l])
        assert int(got["M"][seq, l]) == m, f"{where}: M[{l}] {got['M'][seq, l]} != {m}"
        assert np.array_equal(got["rows"][seq, l, :m], sel.rows[l]), f"{where}: rows of layer {l}"


def host_model_from_device(dev, cfg) -> dict:
    """Bit copy of a ``DeviceModel``'s tensors into the dictionary layout of ``synth.make_model``."""
    return dev.to_host(cfg)


def run_step_pair(sess: Session, frames: np.ndarray, feats: np.ndarray, ids: np.ndarray, params: orc.SelectParams,
                  force_full=False, act_embed: np.ndarray = None, layer_major=False):
    """One control step on both sides with replay: the checker's selection is computed from the
    library's own saved attention (bit-copied) and the checker is fed the library's tokens.

    frames [B, n_cams, H, W, 3] uint8; feats [B, L_v, hidden] bf16 bits; ids [B, n_text] int32.
    With ``act_embed`` ([n_action, hidden] bf16 bits) both sides decode the action chunk in one parallel
    pass instead (vlac_step_chunk / step_chunk); the K/V rows of the chunk are compared as well.
    ``layer_major`` takes the checker's step through ``oracle_compose.step_layer_major`` (same bits, each
    layer's weights widened once per step: for the 32-layer model).
    Returns a dict of per-sequence comparison figures.
    """
    cfg, B = sess.cfg, sess.batch
    gp, keep = gparams(params)
    attn_before = [sess.read_attn(vb.PART_ATTN_PREV, b) for b in range(B)]
    d_frames = torch.from_numpy(frames).to("cuda").contiguous()
    d_feats = vb.upload_bf16(feats)
    d_ids = torch.from_numpy(ids.astype(np.int32)).to("cuda").contiguous()
    tokens = torch.zeros((B, cfg.n_action), dtype=torch.int32, device="cuda")
    logits = torch.zeros((B, cfg.n_action, cfg.vocab), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    d_act = vb.upload_bf16(act_embed) if act_embed is not None else None
    if d_act is not None:
        sess.keep_alive = getattr(sess, "keep_alive", []) + [d_act]      # a captured step may read it again
    with torch.cuda.stream(sess.stream):
        if d_act is None:
            vb.vlac_step(sess.ctx, sess.cache, d_frames, d_feats, d_ids, gp, force_full, tokens, logits)
        else:
            vb.vlac_step_chunk(sess.ctx, sess.cache, d_frames, d_feats, d_ids, gp, force_full, d_act, tokens, logits)
    torch.cuda.synchronize()
    assert vb.vlac_device_error(sess.ctx) == 0
    got_sel = vb.selection_to_host(vb.vlac_selection_view(sess.cache))
    g_tokens, g_logits = tokens.cpu().numpy(), logits.cpu().numpy().astype(np.float64)
    out = []
    for b in range(B):
        oc = sess.ocache[b]
        if oc.warm:
            oc.attn_tv = attn_before[b].astype(np.float64)          # replay: the library's saved scores
        sel = orc.select(cfg, frames[b], oc, params, force_full)
        if oc.warm and not force_full:
            check_selection(got_sel, sel, b, cfg, where=f"seq {b}")
        else:
            assert np.all(got_sel["M"][b] == cfg.seq_len)
        if act_embed is None and layer_major:
            import oracle_compose
            res = oracle_compose.step_layer_major(cfg, sess.model, oc, frames[b], feats[b], ids[b], params,
                                                  forced_tokens=g_tokens[b], force_full=force_full, selection=sel, operands=OPERANDS)
        elif act_embed is None:
            res = orc.step(cfg, sess.model, oc, frames[b], feats[b], ids[b], params, force_full,
                           forced_tokens=g_tokens[b], selection=sel, operands=OPERANDS)
        else:
            res = orc.step_chunk(cfg, sess.model, oc, frames[b], feats[b], ids[b], params, act_embed, force_full,
                                 selection=sel, operands=OPERANDS)
        err = max(rel_err(g_logits[b, i], res.logits[i]) for i in range(cfg.n_action))
        abs_err = float(np.max(np.abs(g_logits[b] - res.logits)))
        # Tokens: identical wherever the checker's top-2 margin exceeds twice the measured logit error.  Below that
        # margin ("guarded") the two may differ, but only as a near-tie: the library's token must then score within
        # the same bound of the checker's best logit ("flipped").  Both counts are reported; the tests bound them.
        guarded = flipped = 0
        for i in range(cfg.n_action):
            same = int(g_tokens[b, i]) == int(res.tokens[i])
            if res.margins[i] > 2.0 * abs_err:
                assert same, f"seq {b} token {i}: {int(g_tokens[b, i])} != {int(res.tokens[i])} at margin {res.margins[i]:.3g}"
            else:
                guarded += 1
                if not same:
                    flipped += 1
                    gap = float(res.logits[i].max() - res.logits[i][int(g_tokens[b, i])])
                    assert gap <= 2.0 * abs_err, f"seq {b} token {i}: the library's token is {gap:.3g} below the best logit"
        g_attn = sess.read_attn(vb.PART_ATTN_PREV, b)
        attn_err = rel_err(g_attn, res.attn_tv)
        attn_err_layers = [rel_err(g_attn[l], res.attn_tv[l]) for l in range(cfg.n_layers)]
        kv_err = 0.0
        if act_embed is not None:
            L, n = cfg.seq_len, cfg.n_action
            for l in range(cfg.n_layers):
                kv_err = max(kv_err, rel_err(sess.read_kv(vb.PART_K, l, b)[L:L + n], oc.K[l][L:L + n]),
                             rel_err(sess.read_kv(vb.PART_V, l, b)[L:L + n], oc.V[l][L:L + n]))
        out.append({"logit_err": err, "abs_err": abs_err, "guarded": guarded, "flipped": flipped, "attn_err": attn_err, "attn_err_layers": attn_err_layers, "kv_err": kv_err,
                    "logit_err_rows": [rel_err(g_logits[b, i], res.logits[i]) for i in range(cfg.n_action)],
                    "margins": res.margins.copy(), "ref_tokens": res.tokens.copy(), "ref_logits": res.logits, "got_logits": g_logits[b],
                    "M": sel.M.copy(), "tokens": g_tokens[b].copy(), "selection": sel})
    return out
