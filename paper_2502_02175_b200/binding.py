"""ctypes binding of ``libvlac.so``: the same names as the C entry points (include/vlac.h).

Argument marshalling only -- every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and streams.  There is no CPU fallback: importing this module
without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvlac.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2502_02175_b200.build` "
        "(the CUDA library is the only implementation; there is no fallback)")
lib = C.CDLL(LIB_PATH)

VLAC_OK = 0
PART_K, PART_V, PART_PREV_FRAME, PART_ATTN_PREV, PART_ATTN_NEXT, PART_WARM, PART_PREV_FRAME_BF16 = range(7)
MAX_LAYERS = 64


class vlac_config(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "hidden", "n_heads", "n_kv_heads", "head_dim", "ffn", "vocab",
                                       "n_cams", "grid", "patch", "n_text_pre", "n_text_post", "n_action")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("max_batch", C.c_int)]


class vlac_layer_w(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g_attn", "g_mlp")]


class vlac_weights(C.Structure):
    _fields_ = [("layers", C.POINTER(vlac_layer_w)), ("embed", C.c_void_p), ("proj", C.c_void_p),
                ("g_final", C.c_void_p), ("lm_head", C.c_void_p), ("rope_cos", C.c_void_p), ("rope_sin", C.c_void_p)]


class vlac_select_params(C.Structure):
    _fields_ = [("tau", C.c_double), ("top_k", C.c_int), ("tau_task", C.c_double), ("task_mode", C.c_int),
                ("k_ent", C.c_double), ("alpha_override", C.POINTER(C.c_double)), ("layer_mask", C.c_ulonglong)]


class vlac_selection(C.Structure):
    _fields_ = [("batch", C.c_int), ("n_layers", C.c_int), ("seq_len", C.c_int), ("n_vision", C.c_int),
                ("M", C.c_void_p), ("rows", C.c_void_p), ("static_mask", C.c_void_p), ("task_mask", C.c_void_p),
                ("final_mask", C.c_void_p), ("sim", C.c_void_p), ("S", C.c_void_p), ("alpha", C.c_void_p)]


EXPORTS = ("vlac_create", "vlac_destroy", "vlac_cache_alloc", "vlac_cache_reset", "vlac_cache_free",
           "vlac_cache_read", "vlac_cache_write", "vlac_select", "vlac_select_bf16", "vlac_select_import", "vlac_layer_forward",
           "vlac_step", "vlac_step_chunk", "vlac_step_pruned", "vlac_selection_view", "vlac_launch_count", "vlac_device_error", "vlac_status_string",
           "vlac_profile", "vlac_profile_read", "vlac_profile_segments", "vlac_greedy_tokens_static",
           "vlac_selftest_wait_expiry")

lib.vlac_status_string.restype = C.c_char_p
lib.vlac_status_string.argtypes = [C.c_int]
lib.vlac_launch_count.restype = C.c_ulonglong
lib.vlac_launch_count.argtypes = [C.c_void_p]
lib.vlac_create.argtypes = [C.POINTER(vlac_config), C.POINTER(vlac_weights), C.POINTER(C.c_void_p)]
lib.vlac_destroy.argtypes = [C.c_void_p]
lib.vlac_cache_alloc.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_void_p)]
lib.vlac_cache_reset.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
lib.vlac_cache_free.argtypes = [C.c_void_p]
lib.vlac_cache_read.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_ulonglong, C.c_void_p]
lib.vlac_cache_write.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_ulonglong, C.c_void_p]
lib.vlac_select.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(vlac_select_params), C.POINTER(vlac_selection), C.c_void_p]
lib.vlac_select_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(vlac_select_params), C.POINTER(vlac_selection), C.c_void_p]
lib.vlac_select_import.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.vlac_layer_forward.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
lib.vlac_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(vlac_select_params), C.c_int,
                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.vlac_step_chunk.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(vlac_select_params), C.c_int,
                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.vlac_step_pruned.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.vlac_selection_view.argtypes = [C.c_void_p, C.POINTER(vlac_selection)]
lib.vlac_device_error.argtypes = [C.c_void_p, C.c_void_p]
lib.vlac_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_uint, C.c_void_p]
lib.vlac_profile.argtypes = [C.c_void_p, C.c_int]
lib.vlac_profile_segments.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.c_int, C.POINTER(C.c_int)]
lib.vlac_greedy_tokens_static.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_longlong, C.c_void_p, C.c_void_p]
lib.vlac_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_ulonglong), C.POINTER(C.c_int)]


class VlacError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib.vlac_status_string(status).decode()} ({status})")


def _check(status: int, where: str) -> None:
    if status != VLAC_OK:
        raise VlacError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def make_config(cfg, max_batch: int = 1) -> vlac_config:
    """``cfg`` is a ``synth.ModelConfig`` (or anything with the same attributes)."""
    return vlac_config(cfg.n_layers, cfg.hidden, cfg.n_heads, cfg.n_heads, cfg.head_dim, cfg.ffn, cfg.vocab,
                       cfg.n_cams, cfg.grid, cfg.patch, cfg.n_text_pre, cfg.n_text_post, cfg.n_action,
                       cfg.rms_eps, cfg.rope_theta, max_batch)


def make_params(tau=0.996, top_k=100, tau_task=0.5, task_mode=0, k_ent=1.0,
                alpha_override: Optional[Sequence[float]] = None, layer_mask: int = 0):
    """Returns (struct, keepalive)."""
    keep = None
    ptr = C.POINTER(C.c_double)()
    if alpha_override is not None:
        keep = (C.c_double * len(alpha_override))(*[float(a) for a in alpha_override])
        ptr = C.cast(keep, C.POINTER(C.c_double))
    return vlac_select_params(tau, top_k, tau_task, task_mode, k_ent, ptr, layer_mask), keep


def upload_bf16(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 patterns -> torch.bfloat16 tensor on the device (bit copy)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device)
    return t.view(torch.bfloat16)


class DeviceModel:
    """Device copies of a ``synth.make_model`` dictionary plus the ``vlac_weights`` struct."""

    def __init__(self, model: Dict[str, object], device="cuda"):
        self.tensors = []
        self.layer_structs = (vlac_layer_w * len(model["layers"]))()
        for i, lw in enumerate(model["layers"]):
            for name, _ in vlac_layer_w._fields_:
                t = upload_bf16(lw[name], device)
                self.tensors.append(t)
                setattr(self.layer_structs[i], name, t.data_ptr())
        self.weights = vlac_weights()
        self.weights.layers = C.cast(self.layer_structs, C.POINTER(vlac_layer_w))
        for name in ("embed", "proj", "g_final", "lm_head"):
            t = upload_bf16(model[name], device)
            self.tensors.append(t)
            setattr(self.weights, name, t.data_ptr())
        for name in ("rope_cos", "rope_sin"):
            t = torch.from_numpy(np.ascontiguousarray(model[name], dtype=np.float32)).to(device)
            self.tensors.append(t)
            setattr(self.weights, name, t.data_ptr())

    def to_host(self, cfg) -> Dict[str, object]:
        """Bit copy of every tensor into the dictionary layout of ``synth.make_model`` (bf16 as uint16 patterns;
        the rotary tables cut to the ``cfg.max_seq`` rows that layout has)."""
        by_ptr = {t.data_ptr(): t for t in self.tensors}

        def bits(ptr):
            t = by_ptr[ptr]
            if t.dtype == torch.bfloat16:
                return t.view(torch.int16).cpu().numpy().view(np.uint16)
            return t.cpu().numpy()

        model = {"layers": [{name: bits(getattr(self.layer_structs[l], name)) for name, _ in vlac_layer_w._fields_}
                            for l in range(cfg.n_layers)]}
        for name in ("embed", "proj", "g_final", "lm_head"):
            model[name] = bits(getattr(self.weights, name))
        for name in ("rope_cos", "rope_sin"):
            model[name] = bits(getattr(self.weights, name))[:cfg.max_seq]
        return model

    @classmethod
    def random(cls, cfg, seed: int, device="cuda") -> "DeviceModel":
        """Random-init weights generated on the device (same distributions as ``synth.make_model``;
        different draws).  For benchmarks where no host copy is needed."""
        from . import synth
        self = cls.__new__(cls)
        self.tensors = []
        gen = torch.Generator(device=device)
        gen.manual_seed(seed)
        shapes = synth.layer_shapes(cfg)

        def mat(shape, std, mean=0.0):
            t = (torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * std + mean).to(torch.bfloat16)
            self.tensors.append(t)
            return t.data_ptr()

        self.layer_structs = (vlac_layer_w * cfg.n_layers)()
        for i in range(cfg.n_layers):
            for name in synth.LAYER_MATRICES:
                setattr(self.layer_structs[i], name, mat(shapes[name], 0.02))
            self.layer_structs[i].g_attn = mat((cfg.hidden,), 0.1, 1.0)
            self.layer_structs[i].g_mlp = mat((cfg.hidden,), 0.1, 1.0)
        self.weights = vlac_weights()
        self.weights.layers = C.cast(self.layer_structs, C.POINTER(vlac_layer_w))
        self.weights.embed = mat((cfg.vocab, cfg.hidden), 0.02)
        self.weights.proj = mat((cfg.hidden, cfg.hidden), 0.02)
        self.weights.g_final = mat((cfg.hidden,), 0.1, 1.0)
        self.weights.lm_head = mat((cfg.vocab, cfg.hidden), 0.02)
        cos, sin = synth.rope_tables(cfg)
        for name, arr in (("rope_cos", cos), ("rope_sin", sin)):
            t = torch.from_numpy(arr).to(device)
            self.tensors.append(t)
            setattr(self.weights, name, t.data_ptr())
        return self


# --------------------------------------------------------------------------- C entry points
def vlac_create(cfg_struct: vlac_config, weights: vlac_weights) -> int:
    out = C.c_void_p()
    _check(lib.vlac_create(C.byref(cfg_struct), C.byref(weights), C.byref(out)), "vlac_create")
    return out.value


def vlac_destroy(ctx: int) -> None:
    _check(lib.vlac_destroy(ctx), "vlac_destroy")


def vlac_cache_alloc(ctx: int, batch: int) -> int:
    out = C.c_void_p()
    _check(lib.vlac_cache_alloc(ctx, batch, C.byref(out)), "vlac_cache_alloc")
    return out.value


def vlac_cache_reset(cache: int, seq: int = -1) -> None:
    _check(lib.vlac_cache_reset(cache, seq, _stream()), "vlac_cache_reset")


def vlac_cache_free(cache: int) -> None:
    _check(lib.vlac_cache_free(cache), "vlac_cache_free")


def vlac_cache_read(cache: int, part: int, seq: int, layer: int, dst: torch.Tensor) -> None:
    assert dst.is_cuda and dst.is_contiguous()
    _check(lib.vlac_cache_read(cache, part, seq, layer, dst.data_ptr(), dst.numel() * dst.element_size(), _stream()),
           "vlac_cache_read")


def vlac_cache_write(cache: int, part: int, seq: int, layer: int, src: torch.Tensor) -> None:
    assert src.is_cuda and src.is_contiguous()
    _check(lib.vlac_cache_write(cache, part, seq, layer, src.data_ptr(), src.numel() * src.element_size(), _stream()),
           "vlac_cache_write")


def vlac_select(ctx: int, cache: int, frames: torch.Tensor, params: vlac_select_params) -> vlac_selection:
    assert frames.is_cuda and frames.dtype == torch.uint8 and frames.is_contiguous()
    out = vlac_selection()
    _check(lib.vlac_select(ctx, cache, frames.data_ptr(), C.byref(params), C.byref(out), _stream()), "vlac_select")
    return out


def vlac_select_bf16(ctx: int, cache: int, frames_bf16: torch.Tensor, params: vlac_select_params) -> vlac_selection:
    assert frames_bf16.is_cuda and frames_bf16.dtype == torch.bfloat16 and frames_bf16.is_contiguous()
    out = vlac_selection()
    _check(lib.vlac_select_bf16(ctx, cache, frames_bf16.data_ptr(), C.byref(params), C.byref(out), _stream()), "vlac_select_bf16")
    return out


def vlac_select_import(ctx: int, cache: int, M: np.ndarray, rows: np.ndarray) -> None:
    M = np.ascontiguousarray(M, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    _check(lib.vlac_select_import(ctx, cache, M.ctypes.data, rows.ctypes.data, _stream()), "vlac_select_import")


def vlac_layer_forward(ctx: int, cache: int, layer: int, hidden: torch.Tensor) -> None:
    assert hidden.is_cuda and hidden.dtype == torch.bfloat16 and hidden.is_contiguous()
    _check(lib.vlac_layer_forward(ctx, cache, layer, hidden.data_ptr(), _stream()), "vlac_layer_forward")


def vlac_step(ctx: int, cache: int, frames: torch.Tensor, vision_feats: torch.Tensor, prompt_ids: torch.Tensor,
              params: Optional[vlac_select_params], force_full: bool, action_tokens: torch.Tensor,
              all_logits: Optional[torch.Tensor] = None, forced_tokens: Optional[torch.Tensor] = None) -> None:
    assert frames.is_cuda and frames.dtype == torch.uint8 and frames.is_contiguous()
    assert vision_feats.is_cuda and vision_feats.dtype == torch.bfloat16 and vision_feats.is_contiguous()
    assert prompt_ids.is_cuda and prompt_ids.dtype == torch.int32 and prompt_ids.is_contiguous()
    assert action_tokens.is_cuda and action_tokens.dtype == torch.int32 and action_tokens.is_contiguous()
    assert all_logits is None or (all_logits.is_cuda and all_logits.dtype == torch.float32 and all_logits.is_contiguous())
    assert forced_tokens is None or (forced_tokens.is_cuda and forced_tokens.dtype == torch.int32)
    _check(lib.vlac_step(ctx, cache, frames.data_ptr(), vision_feats.data_ptr(), prompt_ids.data_ptr(),
                         C.byref(params) if params is not None else None, int(bool(force_full)),
                         action_tokens.data_ptr(), _ptr(all_logits), _ptr(forced_tokens), _stream()), "vlac_step")


def vlac_step_chunk(ctx: int, cache: int, frames: torch.Tensor, vision_feats: torch.Tensor, prompt_ids: torch.Tensor,
                    params: Optional[vlac_select_params], force_full: bool, act_embed: torch.Tensor,
                    action_tokens: torch.Tensor, all_logits: Optional[torch.Tensor] = None) -> None:
    assert frames.is_cuda and frames.dtype == torch.uint8 and frames.is_contiguous()
    assert vision_feats.is_cuda and vision_feats.dtype == torch.bfloat16 and vision_feats.is_contiguous()
    assert prompt_ids.is_cuda and prompt_ids.dtype == torch.int32 and prompt_ids.is_contiguous()
    assert act_embed.is_cuda and act_embed.dtype == torch.bfloat16 and act_embed.is_contiguous()
    assert action_tokens.is_cuda and action_tokens.dtype == torch.int32 and action_tokens.is_contiguous()
    assert all_logits is None or (all_logits.is_cuda and all_logits.dtype == torch.float32 and all_logits.is_contiguous())
    _check(lib.vlac_step_chunk(ctx, cache, frames.data_ptr(), vision_feats.data_ptr(), prompt_ids.data_ptr(),
                               C.byref(params) if params is not None else None, int(bool(force_full)),
                               act_embed.data_ptr(), action_tokens.data_ptr(), _ptr(all_logits), _stream()), "vlac_step_chunk")


def vlac_step_pruned(ctx: int, cache: int, frames: torch.Tensor, vision_feats: torch.Tensor, prompt_ids: torch.Tensor,
                     prune_layer: int, n_keep: int, action_tokens: torch.Tensor, all_logits: Optional[torch.Tensor] = None,
                     forced_tokens: Optional[torch.Tensor] = None) -> None:
    assert frames.is_cuda and frames.dtype == torch.uint8 and frames.is_contiguous()
    assert vision_feats.is_cuda and vision_feats.dtype == torch.bfloat16 and vision_feats.is_contiguous()
    assert prompt_ids.is_cuda and prompt_ids.dtype == torch.int32 and prompt_ids.is_contiguous()
    assert action_tokens.is_cuda and action_tokens.dtype == torch.int32 and action_tokens.is_contiguous()
    assert all_logits is None or (all_logits.is_cuda and all_logits.dtype == torch.float32 and all_logits.is_contiguous())
    _check(lib.vlac_step_pruned(ctx, cache, frames.data_ptr(), vision_feats.data_ptr(), prompt_ids.data_ptr(), int(prune_layer),
                                int(n_keep), action_tokens.data_ptr(), _ptr(all_logits), _ptr(forced_tokens), _stream()), "vlac_step_pruned")


def vlac_selection_view(cache: int) -> vlac_selection:
    out = vlac_selection()
    _check(lib.vlac_selection_view(cache, C.byref(out)), "vlac_selection_view")
    return out


def vlac_launch_count(ctx: int) -> int:
    return int(lib.vlac_launch_count(ctx))


def vlac_device_error(ctx: int) -> int:
    return int(lib.vlac_device_error(ctx, _stream()))


def vlac_selftest_wait_expiry(ctx: int, limit_us: int) -> int:
    """Status of the bounded-wait self-test (VLAC_ERR_TIMEOUT = -5 when the wait gave up as designed)."""
    return int(lib.vlac_selftest_wait_expiry(ctx, int(limit_us), _stream()))


def vlac_profile(ctx: int, enable: bool) -> None:
    _check(lib.vlac_profile(ctx, int(bool(enable))), "vlac_profile")


def vlac_profile_segments(ctx: int):
    """Device ms of the parts of the last profiled step: [select, input rows, prefill, first token, pass 1, ...]."""
    buf = (C.c_double * 16)()
    n = C.c_int()
    _check(lib.vlac_profile_segments(ctx, buf, 16, C.byref(n)), "vlac_profile_segments")
    return [buf[i] for i in range(n.value)]


def vlac_profile_read(ctx: int):
    """(total ms, total weight bytes, launches) of the timed matrix-vector launches."""
    ms, by, n = C.c_double(), C.c_ulonglong(), C.c_int()
    _check(lib.vlac_profile_read(ctx, C.byref(ms), C.byref(by), C.byref(n)), "vlac_profile_read")
    return ms.value, by.value, n.value


def vlac_greedy_tokens_static(logits: torch.Tensor, tokens: torch.Tensor) -> None:
    """Argmax of each row of a 2-D fp32 device tensor into an int32 device tensor, ties to the lower
    index, using only the scratch array built into the library (no allocation; at most 64 rows).
    Meant for callers that may not allocate device memory when they run."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.dim() == 2 and logits.stride(1) == 1
    assert tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous()
    _check(lib.vlac_greedy_tokens_static(logits.data_ptr(), logits.shape[0], logits.shape[1], logits.stride(0),
                                         tokens.data_ptr(), _stream()), "vlac_greedy_tokens_static")


# --------------------------------------------------------------------------- reading views back
_CUDART = None


def _memcpy_d2h(dst: np.ndarray, src_ptr: int) -> None:
    """Blocking device-to-host copy of a library-owned buffer (cudaMemcpy; synchronises)."""
    global _CUDART
    if _CUDART is None:
        name = [n for n in os.listdir(os.path.join(os.path.dirname(torch.__file__), "lib")) if n.startswith("libcudart")]
        _CUDART = C.CDLL(os.path.join(os.path.dirname(torch.__file__), "lib", name[0])) if name else C.CDLL("libcudart.so")
        _CUDART.cudaMemcpy.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_int]
    torch.cuda.current_stream().synchronize()
    rc = _CUDART.cudaMemcpy(dst.ctypes.data, src_ptr, dst.nbytes, 2)
    if rc != 0:
        raise RuntimeError(f"cudaMemcpy failed ({rc})")


def selection_to_host(sel: vlac_selection) -> Dict[str, np.ndarray]:
    """Copy every view of a selection to numpy arrays."""
    B, nl, L, Lv = sel.batch, sel.n_layers, sel.seq_len, sel.n_vision
    out = {
        "M": np.empty((B, nl), np.int32), "rows": np.empty((B, nl, L), np.int32),
        "static_mask": np.empty((B, Lv), np.uint8), "task_mask": np.empty((B, Lv), np.uint8),
        "final_mask": np.empty((B, Lv), np.uint8), "sim": np.empty((B, Lv), np.float64),
        "S": np.empty((B, Lv), np.float64), "alpha": np.empty((B, nl), np.float64),
    }
    for k, arr in out.items():
        _memcpy_d2h(arr, getattr(sel, k))
    return out
